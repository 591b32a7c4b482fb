// Rejection islands (Sec. 3.4, Eq. 8): {I_m} = CC_8(R_X), the 8-connected components of the
// set of positions to redraw, one CTA per image.
//
// The grid of one image (at most kIslandMaxCells positions) lives in shared memory as a
// forest: parent[t] is an earlier raster index of the same island, a root points at itself.
// Horizontal links cost nothing: every position starts out pointing at the first position of
// its run of consecutive R_X bits in the row, found with bit operations on the mask words.
// Only the first position of a run then works: it joins its run with every run of the row
// above that reaches into columns [first - 1, last + 1].  Joining hangs the later root under
// the earlier one with atomicMin, so the root of an island is its first raster position;
// numbering the roots in raster order (a block-wide count) numbers the islands by their
// first position.
#pragma once
#include <cstdint>

namespace mulo {

constexpr int kIslandThreads = 1024;
constexpr int kIslandMaxCells = 16384;

struct IslandArgs {
  int H, W, max_islands;
  const uint32_t* bits;   // [B, H, ceil(W/32)]
  int32_t* labels;        // [B, H, W]
  int32_t* n_islands;     // [B]
  int32_t* rows;          // [B, max_islands, 2] or null
  int32_t* size;          // [B, max_islands] or null
};

// Root of x.  Parents only ever decrease and a root points at itself, so the walk ends.
__device__ __forceinline__ int island_root(const volatile int* parent, int x) {
  int p = parent[x];
  while (p != x) {
    x = p;
    p = parent[x];
  }
  return x;
}

// Joins the islands of a and b.  If another thread re-parents the later root between the
// look-up and the atomicMin, the link it made is kept by carrying on from that parent.
__device__ __forceinline__ void island_join(int* parent, int a, int b) {
  for (;;) {
    a = island_root(parent, a);
    b = island_root(parent, b);
    if (a == b) return;
    if (a < b) {
      const int t = a;
      a = b;
      b = t;
    }
    const int old = atomicMin(&parent[a], b);
    if (old == a) return;
    a = old;
  }
}

__global__ void __launch_bounds__(kIslandThreads) k_islands(IslandArgs a) {
  extern __shared__ int island_smem[];
  const int H = a.H, W = a.W, N = H * W, Ww = (W + 31) / 32, nw = H * Ww;
  int* const parent = island_smem;                                        // [N]
  int* const number = island_smem + N;                                    // [N], roots only
  uint32_t* const word = reinterpret_cast<uint32_t*>(island_smem + 2 * N);   // [nw]
  __shared__ int s_warp[kIslandThreads / 32];
  __shared__ int s_carry;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  for (int w = tid; w < nw; w += kIslandThreads) {
    uint32_t v = a.bits[(size_t)b * nw + w];
    if (w % Ww == Ww - 1 && (W & 31)) v &= (1u << (W & 31)) - 1u;   // bits past the row's end do not count
    word[w] = v;
  }
  if (tid == 0) s_carry = 0;
  __syncthreads();
  // t = i * W + j without an integer division (t < 2^14: the float quotient is off by one at most)
  const float inv_w = 1.0f / (float)W;
  auto split = [&](int t, int& i, int& j) {
    i = (int)((float)t * inv_w);
    j = t - i * W;
    if (j < 0) {
      --i;
      j += W;
    } else if (j >= W) {
      ++i;
      j -= W;
    }
  };
  auto in_rx = [&](int i, int j) -> bool {
    return i >= 0 && j >= 0 && j < W && ((word[i * Ww + (j >> 5)] >> (j & 31)) & 1u);
  };
  // first column of the run of R_X bits that holds (i, j); (i, j) itself is in R_X
  auto run_first = [&](int i, int j) -> int {
    int w = j >> 5;
    uint32_t gaps = ~word[i * Ww + w] & ((1u << (j & 31)) - 1u);   // zeros below j in its word
    while (gaps == 0u && w > 0) {
      --w;
      gaps = ~word[i * Ww + w];
    }
    return gaps ? (w << 5) + 32 - __clz(gaps) : 0;
  };
  // last column of the run that starts at (i, j)
  auto run_last = [&](int i, int j) -> int {
    int w = j >> 5;
    uint32_t gaps = ~word[i * Ww + w] & ~((2u << (j & 31)) - 1u);   // zeros above j in its word
    while (gaps == 0u && w + 1 < Ww) {
      ++w;
      gaps = ~word[i * Ww + w];
    }
    return gaps ? (w << 5) + __ffs(gaps) - 2 : W - 1;
  };
  for (int t = tid; t < N; t += kIslandThreads) {
    int i, j;
    split(t, i, j);
    parent[t] = in_rx(i, j) ? i * W + run_first(i, j) : -1;
  }
  __syncthreads();

  for (int t = tid; t < N; t += kIslandThreads) {
    int i, j;
    split(t, i, j);
    if (i == 0 || !in_rx(i, j) || in_rx(i, j - 1)) continue;   // only the first position of a run works
    const int last = run_last(i, j);
    // runs of the row above inside columns [lo, hi]: one join per run, at its first bit there
    const int lo = j > 0 ? j - 1 : 0, hi = last + 1 < W ? last + 1 : W - 1;
    for (int w = lo >> 5; w <= hi >> 5; ++w) {
      uint32_t up = word[(i - 1) * Ww + w];
      uint32_t below = w > (lo >> 5) ? word[(i - 1) * Ww + w - 1] >> 31 : 0u;   // bit left of this word
      if (w == lo >> 5) up &= ~((1u << (lo & 31)) - 1u);
      if (w == hi >> 5 && (hi & 31) != 31) up &= (2u << (hi & 31)) - 1u;
      uint32_t firsts = up & ~((up << 1) | below);   // first bit, inside the window, of each run
      while (firsts) {
        const int x = (w << 5) + __ffs(firsts) - 1;
        firsts &= firsts - 1u;
        island_join(parent, t, (i - 1) * W + x);
      }
    }
  }
  __syncthreads();
  // first positions of runs point straight at their root (a reader that meets a half-updated
  // chain still walks to the same root); then everybody else, one hop behind
  for (int t = tid; t < N; t += kIslandThreads) {
    int i, j;
    split(t, i, j);
    if (parent[t] >= 0 && !in_rx(i, j - 1)) parent[t] = island_root(parent, t);
  }
  __syncthreads();
  for (int t = tid; t < N; t += kIslandThreads) {
    int i, j;
    split(t, i, j);
    const int q = parent[t];
    if (q >= 0 && in_rx(i, j - 1)) parent[t] = parent[q];
  }
  __syncthreads();

  // number the roots in raster order
  for (int base = 0; base < N; base += kIslandThreads) {
    const int t = base + tid;
    const bool is_root = t < N && parent[t] == t;
    const unsigned roots = __ballot_sync(0xffffffffu, is_root);
    if (lane == 0) s_warp[warp] = __popc(roots);
    __syncthreads();
    // every warp scans the 32 warp counts
    static_assert(kIslandThreads == 1024, "one count per lane");
    const int mine = s_warp[lane];
    int inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += v;
    }
    const int before = s_carry + __shfl_sync(0xffffffffu, inc - mine, warp);
    const int total = __shfl_sync(0xffffffffu, inc, 31);
    if (is_root) number[t] = before + __popc(roots & ((1u << lane) - 1u)) + 1;
    __syncthreads();
    if (tid == 0) s_carry += total;
  }
  __syncthreads();
  const int M = s_carry;
  if (tid == 0) a.n_islands[b] = M;

  const int cap = a.max_islands;
  int32_t* const rows = a.rows ? a.rows + (size_t)b * cap * 2 : nullptr;
  int32_t* const size = a.size ? a.size + (size_t)b * cap : nullptr;
  for (int m = tid; m < cap; m += kIslandThreads) {
    if (rows) {
      rows[2 * m] = m < M ? H : -1;
      rows[2 * m + 1] = -1;
    }
    if (size) size[m] = 0;
  }
  __syncthreads();
  for (int t = tid; t < N; t += kIslandThreads) {
    const int root = parent[t];
    const int m = root >= 0 ? number[root] : 0;
    a.labels[(size_t)b * N + t] = m;
    int i, j;
    split(t, i, j);
    if (m > 0 && m <= cap && !in_rx(i, j - 1)) {   // one contribution per run of the row
      if (rows) {
        atomicMin(&rows[2 * (m - 1)], i);
        atomicMax(&rows[2 * (m - 1) + 1], i);
      }
      if (size) atomicAdd(&size[m - 1], run_last(i, j) - j + 1);
    }
  }
}

// Island schedule (Sec. 3.4: islands redrawn concurrently, a ZipAR-style row window inside an island):
// the sequential step at which each position of R_X is decoded,
//   step(t) = 1 + max(step of the island's earlier positions in the row,
//                     step of the island's positions in the row above up to column col(t) + window - 1).
// Along a row the recurrence s_k = max(s_{k-1} + 1, d_k) has the closed form
// s_k = max_{l <= k} (d_l + k - l), so the positions of a row are independent of one another: one CTA per
// image, one thread per column, the rows in sequence.
struct ScheduleArgs {
  int H, W, window;
  const int32_t* labels;   // [B, H, W]
  int32_t* step;           // [B, H, W]
  int32_t* n_steps;        // [B]
};

constexpr int kScheduleThreads = 256;

__global__ void __launch_bounds__(kScheduleThreads) k_island_schedule(ScheduleArgs a) {
  extern __shared__ int sched_smem[];
  const int H = a.H, W = a.W, b = blockIdx.x, tid = threadIdx.x;
  int* const lab_up = sched_smem;           // labels of row i - 1
  int* const step_up = sched_smem + W;      // steps of row i - 1
  int* const lab = sched_smem + 2 * W;      // labels of row i
  int* const dep = sched_smem + 3 * W;      // d_k of row i: 1 + what the row above demands
  __shared__ int s_max;
  if (tid == 0) s_max = 0;
  const int32_t* labels = a.labels + (size_t)b * H * W;
  int32_t* step = a.step + (size_t)b * H * W;
  int local_max = 0;
  for (int i = 0; i < H; ++i) {
    __syncthreads();   // the previous row's results are in step_up / lab_up
    for (int j = tid; j < W; j += kScheduleThreads) lab[j] = labels[(size_t)i * W + j];
    __syncthreads();
    for (int j = tid; j < W; j += kScheduleThreads) {
      const int m = lab[j];
      int d = 1;
      if (m > 0 && i > 0) {
        // steps grow along a row of an island: its last position at or before column j + window - 1
        for (int jj = min(W - 1, j + a.window - 1); jj >= 0; --jj)
          if (lab_up[jj] == m) {
            d = step_up[jj] + 1;
            break;
          }
      }
      dep[j] = d;
    }
    __syncthreads();
    for (int j = tid; j < W; j += kScheduleThreads) {
      const int m = lab[j];
      int s = 0;
      if (m > 0) {
        int behind = 0;   // k - l: positions of the island between column jj and column j
        for (int jj = j; jj >= 0; --jj)
          if (lab[jj] == m) {
            s = max(s, dep[jj] + behind);
            ++behind;
          }
      }
      step[(size_t)i * W + j] = s;
      local_max = max(local_max, s);
      // becomes the row above (nobody reads step_up / lab_up any more in this row)
      step_up[j] = s;
      lab_up[j] = m;
    }
  }
  atomicMax(&s_max, local_max);
  __syncthreads();
  if (tid == 0) a.n_steps[b] = s_max;
}

}  // namespace mulo
