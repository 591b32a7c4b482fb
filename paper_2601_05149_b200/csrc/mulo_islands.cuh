// Rejection islands (Sec. 3.4, Eq. 8): {I_m} = CC_8(R_X), the 8-connected components of the
// set of positions to redraw, one CTA per image.
//
// The grid of one image (at most kIslandMaxCells positions) lives in shared memory as a
// forest: parent[t] is an earlier raster index of the same island, a root points at itself.
// Every position of R_X is joined with its already-scanned neighbours (west; north, or
// north-west and north-east when north is not in R_X: with north present those two are
// joined to it by their own west/east links).  Joining hangs the later root under the earlier
// one with atomicMin, so the root of an island is its first raster position; numbering the
// roots in raster order (a block-wide count) numbers the islands by their first position.
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

  for (int w = tid; w < nw; w += kIslandThreads) word[w] = a.bits[(size_t)b * nw + w];
  if (tid == 0) s_carry = 0;
  __syncthreads();
  auto in_rx = [&](int i, int j) -> bool {
    return i >= 0 && j >= 0 && j < W && ((word[i * Ww + (j >> 5)] >> (j & 31)) & 1u);
  };
  for (int t = tid; t < N; t += kIslandThreads) parent[t] = in_rx(t / W, t % W) ? t : -1;
  __syncthreads();

  for (int t = tid; t < N; t += kIslandThreads) {
    const int i = t / W, j = t % W;
    if (!in_rx(i, j)) continue;
    if (in_rx(i, j - 1)) island_join(parent, t, t - 1);
    if (in_rx(i - 1, j)) {
      island_join(parent, t, t - W);
    } else {
      if (in_rx(i - 1, j - 1)) island_join(parent, t, t - W - 1);
      if (in_rx(i - 1, j + 1)) island_join(parent, t, t - W + 1);
    }
  }
  __syncthreads();
  // every position points straight at its root (a reader that meets a half-updated chain
  // still walks to the same root)
  for (int t = tid; t < N; t += kIslandThreads)
    if (parent[t] >= 0) parent[t] = island_root(parent, t);
  __syncthreads();

  // number the roots in raster order
  for (int base = 0; base < N; base += kIslandThreads) {
    const int t = base + tid;
    const bool is_root = t < N && parent[t] == t;
    const unsigned roots = __ballot_sync(0xffffffffu, is_root);
    if (lane == 0) s_warp[warp] = __popc(roots);
    __syncthreads();
    int before = s_carry, total = 0;
    for (int w = 0; w < kIslandThreads / 32; ++w) {
      const int c = s_warp[w];
      if (w < warp) before += c;
      total += c;
    }
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
    if (m > 0 && m <= cap) {
      if (rows) {
        atomicMin(&rows[2 * (m - 1)], t / W);
        atomicMax(&rows[2 * (m - 1) + 1], t / W);
      }
      if (size) atomicAdd(&size[m - 1], 1);
    }
  }
}

}  // namespace mulo
