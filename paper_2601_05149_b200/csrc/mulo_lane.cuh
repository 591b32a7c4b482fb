// The fast path of the fused round for rows with top-k on, when the vocabulary splits
// evenly over a CTA's 256 threads (V = 256 * W, W <= 64 ids per thread).
//
// A persistent CTA (256 threads, three per SM) owns a contiguous range of parent (low-res)
// cells.  Per parent it streams the draft row and then its r*r target rows ONCE through a
// two-slot shared-memory ring.  A slot holds one PHASE of a row: a tiled bulk-tensor copy
// (never multicast) brings 32 bytes for every thread -- the next 16 bf16 (8 fp32) ids of
// the 64-id range that thread owns -- of the conditional and of the unconditional row,
// placed with the 32-byte swizzle so that the 128-bit shared loads of a quarter warp hit
// eight different bank groups.  Owning a CONTIGUOUS id range is what keeps the rest cheap:
//
//   dense phase   per element: unpack, CFG mix (packed fp32, one IEEE rounding per step),
//                 compare with a predicted pivot, and a predicated append of the survivor
//                 to the thread's PRIVATE list (a register cursor; no scan, no atomics, no
//                 cross-lane traffic) plus one bit in the thread's 64-bit survivor mask.
//   lists         two threads (t, t + 128) share one column of R rows of a [R][128] array:
//                 one fills it from the top, the other from the bottom, so a column only
//                 overflows when the PAIR holds too many (a binomial tail far thinner than
//                 one thread's), and consecutive lanes hit consecutive banks.
//   selection     exact k-th largest: a 256-bin histogram of the few entries just above
//                 the pivot, the bin that holds the rank, exact ranking of that bin's
//                 entries.  exp() of every candidate is taken once, against a reference
//                 known BEFORE the row starts (the predicted row maximum), so the partition
//                 sum is (all candidates) - (entries below the threshold) and needs no pass
//                 of its own.
//   draws         the residual max(0, p' - q) or the target weights are summed per thread
//                 (the draft row's list of the same thread holds every q it can need, found
//                 by popcount on the two masks), one block scan in double finds the owner
//                 thread of u * total, which walks its own <= 64 ids.
//
// The pivot, the histogram scale and the exp reference of a row are predicted from the
// previous rows of the same kind (running k-th largest, density below it, maximum); a row
// without prediction takes them from the statistics of its first phase.  A row whose
// prediction fails (too few candidates, a full column, rank outside the histogram, a
// maximum far from the reference, too many ties at the threshold) is appended to a list
// that a second launch works off with the general routines, so results never depend on the
// prediction.  Three block barriers per target row, two per draft row.
#pragma once

#include <cuda.h>

#include "mulo_stream.cuh"

namespace mulo {

constexpr int kLThreads = 256;
constexpr int kLWarps = kLThreads / 32;
constexpr int kLStages = 2;
constexpr int kLTile = kLThreads * 32;   // bytes of one tensor's tile: 32 bytes per thread
constexpr int kLSlot = 2 * kLTile;       // conditional + unconditional
constexpr int kLBins = 256;
constexpr int kLSetAside = 64;           // entries of the crossing bin that are ranked exactly
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kMaxRefGap = 8.0f;       // a row whose maximum lies further from the exp reference leaves the fast path

struct LaneArgs {
  DevParams P;
  const char* cond;
  const char* uncond;
  const char* draft;
  const int32_t* draft_tok_lo;
  float* p_tok;
  float* q_tok;
  float* accept_prob;
  uint8_t* flags;
  int32_t* cand_res;
  int32_t* cand_tgt;
  uint32_t* dev_status;
  int32_t* fail_list;
  int n_parents;
  int W;            // ids per thread = V / 256
  int n_ph;         // phases per row = W / (ids per 32 bytes)
  int R;            // rows of a list column (shared by threads t and t + 128)
  int margin;       // candidates aimed for beyond k
  float a_theta;    // Phi^-1(1 - k/V)
  float a_boot;     // Phi^-1(1 - (k + bootstrap margin)/V)
  float a_max;      // Phi^-1(1 - 1/(2V)): where a normal row's maximum is expected
};

// running prediction for one kind of row (draft / target), per CTA
struct LanePredictor {
  int have;
  float theta, rho, mx;       // running k-th largest, density below it, row maximum
  float pivot, inv_w, ref;    // what the next row starts from (valid while have != 0)
  float shift, step;          // bootstrap adaptation, as in the general streaming kernel
  int dir;
};

struct LaneCursor {            // next item to request into a ring slot
  int left;                    // items still to request into this slot
  int ph, j;                   // phase within the row, row within the parent (0 = draft row)
  int parent, b, ca, cc;
};

// Selection scratch of one row.  Two copies, used by rows of alternating parity: what a row adds
// into (histogram, set-aside list, per-warp partials) is reset / rewritten two rows later, with
// at least two block barriers in between, so no reader of row i can meet a writer of row i + 2.
struct LaneSel {
  unsigned hist[kLBins];
  float sa_z[kLSetAside];
  float sa_e[kLSetAside];
  unsigned n_sa;
  unsigned overflow;
  int w_n[kLWarps];
  float w_max[kLWarps];
  double w_e[kLWarps];
  double w_excl[kLWarps];
};

struct LanePrep {              // per target row, written by two threads before the row's first barrier
  uint32_t rnd[3];
  float z_tok;
  double e_tok;
  uint32_t raw_c, raw_u;       // landing place of the asynchronous copies of the logit words of x~
};

struct LaneSmem {
  uint64_t full[kLStages];
  unsigned done[kLStages];
  LaneCursor cursor[kLStages];
  LaneSel sel[2];
  LanePrep prep[2];
  double w_tot[2][kLWarps];    // block scan of a draw; consecutive draws alternate
  float red[kLWarps][2];
  unsigned char cnt[kLThreads];
  LanePredictor pred[2];
  double q_tok;                // of the current parent
  uint32_t raw_q;              // landing place of the draft logit word of x~
  int tok[2];                  // the draft token of the parent in work / of the next one
};

__device__ __forceinline__ void tma_tile_3d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"((uint64_t)tm), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(bar))
      : "memory");
}
// Bounded wait on a ring slot.  The hint lets the hardware suspend the warp for up to about a
// microsecond per try instead of spinning through the issue slots; after 2^21 tries (seconds) the
// wait gives up and raises the time-out bit.
__device__ __forceinline__ bool mbar_try_wait_hint(uint64_t* bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(ns)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void lane_wait(uint64_t* bar, uint32_t parity, uint32_t* dev_status) {
#pragma unroll 1
  for (uint32_t it = 0; it < (1u << 21); ++it)
    if (mbar_try_wait_hint(bar, parity, 1000u)) return;
  atomicOr(dev_status, MULO_DEV_TIMEOUT);
}
// 4-byte asynchronous global -> shared copy (no register holds the value while it is in flight)
__device__ __forceinline__ void cp_async4(void* dst_smem, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// the 32-bit word that holds logit `at` of a tensor, and the logit's value out of that word
template <bool BF16>
__device__ __forceinline__ const void* logit_word(const char* base, size_t at) {
  return base + ((at * (BF16 ? 2 : 4)) & ~(size_t)3);
}
template <bool BF16>
__device__ __forceinline__ float logit_of_word(uint32_t w, size_t at) {
  if (!BF16) return __uint_as_float(w);
  return __uint_as_float((at & 1) ? (w & 0xffff0000u) : (w << 16));
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ float lds_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts_f32(uint32_t addr, float v) {
  asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
// 2^t by the special-function unit (relative error about 2^-22)
__device__ __forceinline__ float ex2f(float t) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(t));
  return r;
}

// Appends z to a thread's list if z >= pivot, without a branch: the store is unconditional (a
// value below the pivot lands in the next free row and is overwritten by the next survivor, or
// never read), the cursor steps -- clamped at `lim` -- and the mask gains the bit under a select.
template <int STEP, int BIT>
__device__ __forceinline__ void lane_put(float z, float pivot, uint32_t& cur, uint32_t lim, uint32_t& m) {
  const bool p = z >= pivot;
  sts_f32(cur, z);
  const uint32_t nxt = STEP > 0 ? min(cur + (uint32_t)STEP, lim) : max(cur - (uint32_t)(-STEP), lim);
  cur = p ? nxt : cur;
  m |= p ? (1u << BIT) : 0u;
}

template <int J>
__device__ __forceinline__ uint32_t word_of(const uint4& v) {
  return J == 0 ? v.x : J == 1 ? v.y : J == 2 ? v.z : v.w;
}

// Two ids of a phase: word J of 16-byte piece I of the thread's 32 bytes.  bf16: one word of the
// conditional (and unconditional) row holds both; fp32: words 2J and 2J + 1 of piece I hold them
// (J < 2).  Pre-processing as the definition says (d = c - u; v = fma(s, d, u); z = v * invT, each
// one fp32 rounding; two ids per instruction), then the two appends.
template <bool BF16, bool ROW_U, bool SCALE, int STEP, int I, int J>
__device__ __forceinline__ void lane_pair(const uint4 (&c)[2], const uint4 (&u)[2], uint64_t s2, uint64_t t2,
                                          float pivot, uint32_t& cur, uint32_t lim, uint32_t& m) {
  uint64_t v, un;
  if (BF16) {
    const uint32_t cw = word_of<J>(c[I]);
    v = pack2(bf16_lo(cw), bf16_hi(cw));
    if (ROW_U) {
      const uint32_t uw = word_of<J>(u[I]);
      un = pack2(bf16_lo(uw), bf16_hi(uw));
    }
  } else {
    v = pack2(__uint_as_float(word_of<(2 * J) & 3>(c[I])), __uint_as_float(word_of<(2 * J + 1) & 3>(c[I])));
    if (ROW_U) un = pack2(__uint_as_float(word_of<(2 * J) & 3>(u[I])), __uint_as_float(word_of<(2 * J + 1) & 3>(u[I])));
  }
  if (ROW_U) v = fma2(s2, sub2(v, un), un);
  if (SCALE) v = mul2(v, t2);
  float z0, z1;
  unpack2(v, z0, z1);
  constexpr int bit = BF16 ? I * 8 + J * 2 : I * 4 + J * 2;
  lane_put<STEP, bit>(z0, pivot, cur, lim, m);
  lane_put<STEP, bit + 1>(z1, pivot, cur, lim, m);
}

// One phase of a row for one thread: the 32 bytes (16 bf16 / 8 fp32 ids) of the conditional row at
// `sb` (and of the unconditional row one tile further); survivors z >= pivot are appended at `cur`
// (stepping by STEP bytes, clamped at `lim`) and marked in the returned mask.
template <bool BF16, bool ROW_U, bool SCALE, int STEP>
__device__ __forceinline__ uint32_t lane_dense(uint32_t sb, uint32_t sw, float s, float invT, float pivot,
                                               uint32_t& cur, uint32_t lim) {
  // the second 16 bytes are loaded after the first have been worked off: half as many live registers
  uint4 c[2], u[2];
  c[0] = lds128(sb + (sw << 4));
  u[0] = ROW_U ? lds128(sb + kLTile + (sw << 4)) : make_uint4(0, 0, 0, 0);
  const uint64_t s2 = pack2(s, s), t2 = pack2(invT, invT);
  uint32_t m = 0;
  lane_pair<BF16, ROW_U, SCALE, STEP, 0, 0>(c, u, s2, t2, pivot, cur, lim, m);
  lane_pair<BF16, ROW_U, SCALE, STEP, 0, 1>(c, u, s2, t2, pivot, cur, lim, m);
  if (BF16) {
    lane_pair<BF16, ROW_U, SCALE, STEP, 0, 2>(c, u, s2, t2, pivot, cur, lim, m);
    lane_pair<BF16, ROW_U, SCALE, STEP, 0, 3>(c, u, s2, t2, pivot, cur, lim, m);
  }
  c[1] = lds128(sb + ((1u ^ sw) << 4));
  u[1] = ROW_U ? lds128(sb + kLTile + ((1u ^ sw) << 4)) : make_uint4(0, 0, 0, 0);
  lane_pair<BF16, ROW_U, SCALE, STEP, 1, 0>(c, u, s2, t2, pivot, cur, lim, m);
  lane_pair<BF16, ROW_U, SCALE, STEP, 1, 1>(c, u, s2, t2, pivot, cur, lim, m);
  if (BF16) {
    lane_pair<BF16, ROW_U, SCALE, STEP, 1, 2>(c, u, s2, t2, pivot, cur, lim, m);
    lane_pair<BF16, ROW_U, SCALE, STEP, 1, 3>(c, u, s2, t2, pivot, cur, lim, m);
  }
  return m;
}

template <bool BF16, bool HAS_U>
__global__ void __launch_bounds__(kLThreads, 3)
    k_round_lane(const __grid_constant__ LaneArgs a, const __grid_constant__ CUtensorMap tm_c,
                 const __grid_constant__ CUtensorMap tm_u, const __grid_constant__ CUtensorMap tm_q) {
  constexpr int esz = BF16 ? 2 : 4;
  constexpr int IDS = 32 / esz;   // ids per thread per phase
  __shared__ LaneSmem sm;
  extern __shared__ __align__(128) unsigned char dyn[];
  const DevParams& P = a.P;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int p_begin = (int)(((long long)a.n_parents * blockIdx.x) / gridDim.x);
  const int p_end = (int)(((long long)a.n_parents * (blockIdx.x + 1)) / gridDim.x);
  if (p_end <= p_begin) return;
  const int rr = P.r * P.r, rows_per_parent = 1 + rr;
  const int R = a.R, W = a.W, n_ph = a.n_ph;
  const bool scale = P.invT != 1.0f;
  const int N = P.H * P.W;

  // ---- this thread's places in shared memory
  // (the swizzle works on address bits 4 and 7: the ring starts on a 256-byte boundary)
  const uint32_t ring = (smem_u32(dyn) + 255u) & ~255u;
  // A list column (R rows of 512 bytes; lane l of a warp sits in bank l) belongs to threads t and
  // t + 128 and holds four stacks: the draft row's entries of t from row 0 upwards and of t + 128
  // from row R - 1 downwards (fixed while the parent's children are verified), and between them the
  // current target row's entries of the two threads, again growing towards each other.  A stack is
  // clamped at the first row of the stack it grows towards, so it can never reach the draft entries
  // of the other thread; whether two stacks met is checked from the four counts.
  const bool up = tid < kLThreads / 2;
  const int step = up ? 512 : -512;
  const uint32_t col = ring + kLStages * kLSlot + (uint32_t)(tid & 127) * 4u;
  const uint32_t q_base = col + (up ? 0u : (uint32_t)(R - 1) * 512u);
  const uint32_t q_lim = col + (up ? (uint32_t)(R - 1) * 512u : 0u);   // the partner's first draft row
  const uint32_t sw = ((uint32_t)tid >> 2) & 1u;           // 32-byte swizzle: address bit 4 ^= bit 7
  const uint32_t my_off = (uint32_t)tid * 32u;

  if (tid == 0) {
    for (int s = 0; s < kLStages; ++s) {
      mbar_init(&sm.full[s], 1);
      sm.done[s] = 0;
    }
    mbar_fence_init();
    for (int s = 0; s < 2; ++s) {
      sm.sel[s].n_sa = 0;
      sm.sel[s].overflow = 0;
      LanePredictor& pr = sm.pred[s];
      pr.have = 0;
      pr.theta = 0.f; pr.rho = 1.f; pr.mx = 0.f;
      pr.pivot = 0.f; pr.inv_w = 0.f; pr.ref = 0.f;
      pr.shift = 0.f; pr.step = 0.f; pr.dir = 0;
    }
  }
  sm.sel[0].hist[tid] = 0;
  sm.sel[1].hist[tid] = 0;
  __syncthreads();

  // ---- the ring: items in the order they are consumed; the warp that is last out of a
  //      slot requests the item kLStages further on into it
  auto cursor_advance = [&](LaneCursor& c) {
    if (++c.ph == n_ph) {
      c.ph = 0;
      if (++c.j == rows_per_parent) {
        c.j = 0;
        ++c.parent;
        if (++c.cc == P.w) {
          c.cc = 0;
          if (++c.ca == P.h) {
            c.ca = 0;
            ++c.b;
          }
        }
      }
    }
  };
  auto cursor_issue = [&](const LaneCursor& c, int slot) {
    const uint32_t dst = ring + (uint32_t)slot * kLSlot;
    if (c.j == 0) {
      mbar_expect_tx(&sm.full[slot], kLTile);
      tma_tile_3d(dst, &tm_q, IDS * c.ph, 0, c.parent, &sm.full[slot]);
    } else {
      const int child = c.j - 1;
      const int row = c.b * N + (c.ca * P.r + child / P.r) * P.W + c.cc * P.r + child % P.r;
      mbar_expect_tx(&sm.full[slot], HAS_U ? kLSlot : kLTile);
      tma_tile_3d(dst, &tm_c, IDS * c.ph, 0, row, &sm.full[slot]);
      if (HAS_U) tma_tile_3d(dst + kLTile, &tm_u, IDS * c.ph, 0, row, &sm.full[slot]);
    }
  };
  if (tid == 0) {
    const int total = (p_end - p_begin) * rows_per_parent * n_ph;
    const int hw = P.h * P.w;
    LaneCursor cur;
    cur.ph = 0; cur.j = 0; cur.parent = p_begin; cur.left = 0;
    cur.b = p_begin / hw; cur.ca = (p_begin % hw) / P.w; cur.cc = (p_begin % hw) % P.w;
    for (int s = 0; s < kLStages; ++s) {
      if (s < total) cursor_issue(cur, s);
      LaneCursor nxt = cur;
      for (int k = 0; k < kLStages; ++k) cursor_advance(nxt);
      nxt.left = total > s + kLStages ? (total - s - 1) / kLStages : 0;
      sm.cursor[s] = nxt;
      cursor_advance(cur);
    }
  }
  int rs = 0;   // slots consumed so far: bit 0 = the slot to read next, bit 1 = its phase
#define rslot (rs & 1)
#define rphase ((uint32_t)(rs >> 1) & 1u)
  static_assert(kLStages == 2, "the packed ring state assumes two slots");
  auto release_slot = [&]() {
    __syncwarp();
    if (lane == 0) {
      __threadfence_block();
      const unsigned old = atomicAdd(&sm.done[rslot], 1u);
      if (old == (unsigned)kLWarps - 1u) {
        sm.done[rslot] = 0;
        __threadfence_block();
        LaneCursor cur = sm.cursor[rslot];
        if (cur.left > 0) {
          cursor_issue(cur, rslot);
          --cur.left;
#pragma unroll
          for (int k = 0; k < kLStages; ++k) cursor_advance(cur);
          sm.cursor[rslot] = cur;
        }
      }
    }
    ++rs;
  };
  auto skip_row = [&]() {
    for (int ph = 0; ph < n_ph; ++ph) {
      lane_wait(&sm.full[rslot], rphase, a.dev_status);
      release_slot();
    }
  };

  // ---- pivot, histogram scale and exp reference of the next row of a kind
  auto choose_pivot = [&](int kind, auto row_u_tag, float& pivot, float& inv_w, float& ref) {
    constexpr bool ROW_U = decltype(row_u_tag)::value;
    const LanePredictor pr = sm.pred[kind];
    if (pr.have) {   // block-uniform
      pivot = pr.pivot;
      inv_w = pr.inv_w;
      ref = pr.ref;
      return;
    }
    // no prediction: mean and spread of the row's first phase (every thread's first ids: an
    // even sample of the row), assuming a normal shape; the slot is read again by the dense pass
    lane_wait(&sm.full[rslot], rphase, a.dev_status);
    const uint32_t sb = ring + (uint32_t)rslot * kLSlot + my_off;
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const uint4 c = lds128(sb + (((uint32_t)i ^ sw) << 4));
      uint4 u = make_uint4(0, 0, 0, 0);
      if (ROW_U) u = lds128(sb + kLTile + (((uint32_t)i ^ sw) << 4));
      const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, uw[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (BF16) {
          const float z0 = mix_logit(bf16_lo(cw[j]), bf16_lo(uw[j]), ROW_U, P.cfg_scale, P.invT);
          const float z1 = mix_logit(bf16_hi(cw[j]), bf16_hi(uw[j]), ROW_U, P.cfg_scale, P.invT);
          s1 += z0 + z1;
          s2 += z0 * z0 + z1 * z1;
        } else {
          const float z0 = mix_logit(__uint_as_float(cw[j]), __uint_as_float(uw[j]), ROW_U, P.cfg_scale, P.invT);
          s1 += z0;
          s2 += z0 * z0;
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      s1 += __shfl_xor_sync(kFull, s1, o);
      s2 += __shfl_xor_sync(kFull, s2, o);
    }
    if (lane == 0) {
      sm.red[warp][0] = s1;
      sm.red[warp][1] = s2;
    }
    __syncthreads();
    double S1 = 0.0, S2 = 0.0;
#pragma unroll
    for (int w = 0; w < kLWarps; ++w) {
      S1 += (double)sm.red[w][0];
      S2 += (double)sm.red[w][1];
    }
    __syncthreads();
    const float cnt = (float)(kLThreads * IDS);
    const float mean = (float)(S1 / cnt);
    const float sd = sqrtf(fmaxf((float)(S2 / cnt) - mean * mean, 1e-20f));
    const float d = fmaxf((a.a_theta - a.a_boot) * sd, 1e-20f);
    pivot = mean + (a.a_boot + pr.shift) * sd;
    inv_w = (float)kLBins / (3.0f * d);
    ref = mean + a.a_max * sd;
  };

  // ---- a row through the ring into this thread's list; returns the entry count
  auto stream_row = [&](auto row_u_tag, uint32_t base, uint32_t lim, float pivot, uint32_t& m_lo, uint32_t& m_hi) -> int {
    constexpr bool ROW_U = decltype(row_u_tag)::value;
    uint32_t cur = base;
    m_lo = 0;
    m_hi = 0;
#pragma unroll 1
    for (int ph = 0; ph < n_ph; ++ph) {
      lane_wait(&sm.full[rslot], rphase, a.dev_status);
      const uint32_t sb = ring + (uint32_t)rslot * kLSlot + my_off;
      uint32_t m;
      // the four variants differ in compile-time constants only; the branch is warp-uniform
      if (up) {
        m = scale ? lane_dense<BF16, ROW_U, true, 512>(sb, sw, P.cfg_scale, P.invT, pivot, cur, lim)
                  : lane_dense<BF16, ROW_U, false, 512>(sb, sw, P.cfg_scale, P.invT, pivot, cur, lim);
      } else {
        m = scale ? lane_dense<BF16, ROW_U, true, -512>(sb, sw, P.cfg_scale, P.invT, pivot, cur, lim)
                  : lane_dense<BF16, ROW_U, false, -512>(sb, sw, P.cfg_scale, P.invT, pivot, cur, lim);
      }
      release_slot();
      const int bit0 = ph * IDS;
      if (bit0 < 32) m_lo |= m << bit0;
      else m_hi |= m << (bit0 - 32);
    }
    return up ? (int)((cur - base) >> 9) : (int)((base - cur) >> 9);
  };

  // ---- pass 1 over the thread's own entries: exp against the reference, maximum, histogram of
  //      the low end; per-warp partial results for the block
  auto pass_one = [&](LaneSel& sel, uint32_t base, int n, float pivot, float inv_w, float c0, uint32_t& lowm) {
    const float hoff = -pivot * inv_w;
    float mx = -INFINITY, s_all = 0.f;
    lowm = 0;
    uint32_t ad = base;
#pragma unroll 2
    for (int i = 0; i < n; ++i, ad += step) {
      const float z = lds_f32(ad);
      mx = fmaxf(mx, z);
      s_all += ex2f(fmaf(z, kLog2e, c0));
      // (a column whose stacks have met holds entries from below the pivot until the row is
      // given up after the next barrier: the unsigned compare keeps their bins out of range)
      const unsigned bin = (unsigned)(int)fmaf(z, inv_w, hoff);
      if (bin < (unsigned)kLBins) {
        atomicAdd(&sel.hist[bin], 1u);
        lowm |= 1u << (i & 31);
      }
    }
    sm.cnt[tid] = (unsigned char)n;
    const int nsum = __reduce_add_sync(kFull, n);
    const unsigned mk = __reduce_max_sync(kFull, float_key(mx));
    const double es = warp_sum((double)s_all);
    if (lane == 0) {
      sel.w_n[warp] = nsum;
      sel.w_max[warp] = key_float(mk);
      sel.w_e[warp] = es;
    }
  };

  struct Sel {
    int n, bstar, want, cum, reason;
    float mx;
  };
  // after the barrier that follows pass_one (every warp computes the same)
  auto locate_bin = [&](LaneSel& sel, Sel& s, float ref, int rows) -> bool {
    int n = 0;
    float mx = -INFINITY;
#pragma unroll
    for (int w = 0; w < kLWarps; ++w) {
      n += sel.w_n[w];
      mx = fmaxf(mx, sel.w_max[w]);
    }
    s.n = n;
    s.mx = mx;
    s.reason = 0;
    // the two stacks that grow towards each other must not (nearly) fill the `rows` they share;
    // the bit mask of a thread's low entries covers 32 entries
    const int mine_n = sm.cnt[tid], other_n = sm.cnt[tid ^ 128];
    if (__any_sync(kFull, mine_n + other_n >= rows - 1 || mine_n > 32) && lane == 0) sel.overflow = 1;
    if (n < P.top_k) {
      s.reason = 2;
      return false;
    }
    if (!(fabsf(mx - ref) <= kMaxRefGap)) {
      s.reason = 5;
      return false;
    }
    const int rank = n - P.top_k + 1;   // 1-based rank from the bottom of the k-th largest
    constexpr int PER = kLBins / 32;
    unsigned h[PER];
    unsigned mine = 0;
#pragma unroll
    for (int b = 0; b < PER; ++b) {
      h[b] = sel.hist[lane * PER + b];
      mine += h[b];
    }
    unsigned inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned t = __shfl_up_sync(kFull, inc, o);
      if (lane >= o) inc += t;
    }
    const unsigned owner_mask = __ballot_sync(kFull, inc >= (unsigned)rank);
    if (owner_mask == 0) {
      s.reason = 3;
      return false;
    }
    const int owner = __ffs(owner_mask) - 1;
    unsigned cum = inc - mine, in_bin = 0;
    int bstar = -1;
#pragma unroll
    for (int b = 0; b < PER; ++b) {
      if (bstar < 0) {
        if (cum + h[b] >= (unsigned)rank) {
          bstar = lane * PER + b;
          in_bin = h[b];
        } else {
          cum += h[b];
        }
      }
    }
    s.bstar = __shfl_sync(kFull, bstar, owner);
    s.cum = (int)__shfl_sync(kFull, cum, owner);
    in_bin = __shfl_sync(kFull, in_bin, owner);
    s.want = rank - s.cum;
    if (in_bin > (unsigned)kLSetAside) {
      s.reason = 4;
      return false;
    }
    return true;
  };

  // between the first and the second barrier: the thread's low entries once more -- those below the
  // crossing bin leave the partition sum, those inside it are set aside to be ranked exactly
  auto set_aside = [&](LaneSel& sel, uint32_t base, uint32_t lowm, float pivot, float inv_w, float c0, int bstar) {
    const float hoff = -pivot * inv_w;
    float excl = 0.f;
    while (lowm) {
      const int i = __ffs(lowm) - 1;
      lowm &= lowm - 1;
      const float z = lds_f32(base + (uint32_t)(i * step));
      const int bin = (int)fmaf(z, inv_w, hoff);
      const float e = ex2f(fmaf(z, kLog2e, c0));
      if (bin < bstar) excl += e;
      else if (bin == bstar) {
        const unsigned at = atomicAdd(&sel.n_sa, 1u);
        if (at < (unsigned)kLSetAside) {
          sel.sa_z[at] = z;
          sel.sa_e[at] = e;
        }
      }
    }
    const double ex = warp_sum((double)excl);
    if (lane == 0) sel.w_excl[warp] = ex;
  };

  // after the second barrier: the exact k-th largest value, the number of entries >= it and the
  // partition sum (every thread computes the same from shared data)
  auto finish_selection = [&](LaneSel& sel, const Sel& s, float& theta, int& n_ge, double& Z) -> bool {
    const int mcount = (int)sel.n_sa;   // <= kLSetAside: locate_bin checked the bin's size
    float th = 0.f;
    int less_at = 0;
    bool hit = false;
    for (int i = lane; i < mcount; i += 32) {
      const float vi = sel.sa_z[i];
      int less = 0, leq = 0;
      for (int jj = 0; jj < mcount; ++jj) {
        const float vj = sel.sa_z[jj];
        less += vj < vi;
        leq += vj <= vi;
      }
      if (less < s.want && s.want <= leq) {
        th = vi;
        less_at = less;
        hit = true;
      }
    }
    const unsigned hm = __ballot_sync(kFull, hit);
    if (hm == 0) return false;   // cannot happen: the bin holds the rank
    const int src = __ffs(hm) - 1;
    th = __shfl_sync(kFull, th, src);
    less_at = __shfl_sync(kFull, less_at, src);
    double z = 0.0;
#pragma unroll
    for (int w = 0; w < kLWarps; ++w) z += sel.w_e[w] - sel.w_excl[w];
    // the bin's entries below theta.  The slots were handed out by atomics in no fixed order, but
    // the sum does not depend on it: the entries of one histogram bin share their exponent (or
    // differ by one), so adding up to 64 fp32 values of that kind in double is exact.
    double below = 0.0;
    for (int i = 0; i < mcount; ++i)
      if (sel.sa_z[i] < th) below += (double)sel.sa_e[i];
    Z = z - below;
    theta = th;
    n_ge = s.n - s.cum - less_at;
    return true;
  };

  auto learn = [&](int kind, bool ok, int reason, float theta, float pivot, int n, int n_ge, float mx) {
    LanePredictor pr = sm.pred[kind];
    if (!ok) {
      pr.have = 0;
      const int dir = reason == 2 ? -1 : (reason == 1 || reason == 3) ? 1 : 0;
      if (dir != 0) {
        const float unit = 0.5f * (a.a_theta - a.a_boot);
        if (pr.dir == 0) pr.step = unit;
        else if (pr.dir == dir) pr.step = fminf(2.0f * pr.step, 64.0f * unit);
        else pr.step = fmaxf(0.5f * pr.step, 0.25f * unit);
        pr.shift += (float)dir * pr.step;
        pr.dir = dir;
      }
    } else {
      pr.dir = 0;
      const int below = n - n_ge;   // candidates in [pivot, theta)
      float rho = pr.rho;
      bool rho_ok = pr.have != 0;
      if (theta > pivot && below >= 16) {
        const float r_new = (float)below / (theta - pivot);
        rho = pr.have ? pr.rho + 0.25f * (r_new - pr.rho) : r_new;
        rho_ok = true;
      }
      if (!rho_ok) {
        pr.have = 0;
      } else {
        pr.theta = pr.have ? pr.theta + 0.25f * (theta - pr.theta) : theta;
        pr.mx = pr.have ? pr.mx + 0.25f * (mx - pr.mx) : mx;
        pr.rho = rho;
        pr.have = 1;
        const float d = (float)a.margin / rho;
        pr.pivot = pr.theta - d;
        pr.inv_w = (float)kLBins / (3.0f * d);
        pr.ref = pr.mx;
      }
    }
    sm.pred[kind] = pr;
  };

  auto count_failure = [&](int reason) {   // one thread
    if (reason < 1 || reason > 4) return;
    const int slot = reason == 1 ? kCntListFull : reason == 2 ? kCntTooFew : reason == 3 ? kCntAboveRange : kCntCrowdedBin;
    atomicAdd(a.dev_status + slot, 1u);
  };
  auto defer = [&](size_t g) {   // one thread: position g goes to the general routines
    const unsigned at = atomicAdd(a.dev_status + kFailCount, 1u);
    a.fail_list[at] = (int32_t)g;
    atomicAdd(a.dev_status + kCntRows, 1u);
  };
  // After a row's FIRST barrier: zero the other copy, which the next row adds into.  Its last
  // readers (the previous row, after that row's second barrier) have all arrived at this row's
  // first barrier, and the next row's additions come after this row's second barrier.
  auto reset_selection = [&](LaneSel& sel) {
    sel.hist[tid] = 0;
    if (tid == 0) {
      sel.n_sa = 0;
      sel.overflow = 0;
    }
  };

  uint32_t dm_lo = 0, dm_hi = 0;   // survivor mask of the parent's draft row (this thread's ids)
  int nq = 0, nq_other = 0;        // draft entries of this thread and of the thread it shares the column with
  int rowi = 0;                    // rows done by this CTA (its parity selects the scratch copies)

  if (tid == kLThreads - 1) sm.tok[p_begin & 1] = __ldg(a.draft_tok_lo + p_begin);
  for (int parent = p_begin; parent < p_end; ++parent) {
    // position of the parent's first child: image pb, raster index t0 within the image
    int pb, t0;
    {
      const int hw = P.h * P.w;
      pb = parent / hw;
      const int rem = parent - pb * hw, pca = rem / P.w, pcc = rem - pca * P.w;
      t0 = pca * P.r * P.W + pcc * P.r;
    }
    bool q_ok;
    // ------------------------------------------------------------ draft row
    {
      LaneSel& sel = sm.sel[rowi & 1];
      ++rowi;
      float pivot, inv_w, ref;
      choose_pivot(0, std::false_type{}, pivot, inv_w, ref);
      const float c0 = -ref * kLog2e;
      if (tid == kLThreads - 1) {
        // the draft logit of x~ and the next parent's token: requested now, read after the row
        cp_async_wait_all();
        const int tok = checked_token(sm.tok[parent & 1], P.V, a.dev_status);
        sm.tok[parent & 1] = tok;
        cp_async4(&sm.raw_q, logit_word<BF16>(a.draft, (size_t)parent * P.V + (size_t)tok));
        if (parent + 1 < p_end) cp_async4(&sm.tok[(parent + 1) & 1], a.draft_tok_lo + parent + 1);
      }
      nq = stream_row(std::false_type{}, q_base, q_lim, pivot, dm_lo, dm_hi);
      uint32_t lowm;
      pass_one(sel, q_base, nq, pivot, inv_w, c0, lowm);
      __syncthreads();   // ---- barrier 1
      reset_selection(sm.sel[rowi & 1]);
      Sel s;
      bool ok = locate_bin(sel, s, ref, R);
      nq_other = sm.cnt[tid ^ 128];
      if (ok) set_aside(sel, q_base, lowm, pivot, inv_w, c0, s.bstar);
      __syncthreads();   // ---- barrier 2
      float theta = 0.f;
      int n_ge = 0;
      double Zq = 1.0;
      if (ok && sel.overflow) {
        ok = false;
        s.reason = 1;
      }
      if (ok) ok = finish_selection(sel, s, theta, n_ge, Zq);
      if (ok && !(Zq > 0.0 && Zq < 1e300)) ok = false;
      if (ok) {
        // q in place of z: q(x) = [z >= theta] exp(z - ref) / Z_q, the fp32 product of e and 1/Z_q
        const float invZq = (float)(1.0 / Zq);
        uint32_t ad = q_base;
#pragma unroll 2
        for (int i = 0; i < nq; ++i, ad += step) {
          const float z = lds_f32(ad);
          const float e = ex2f(fmaf(z, kLog2e, c0));
          sts_f32(ad, z >= theta ? __fmul_rn(e, invZq) : 0.f);
        }
      }
      if (tid == kLThreads - 1) {
        if (ok) {
          cp_async_wait_all();
          const size_t at = (size_t)parent * P.V + (size_t)sm.tok[parent & 1];
          const float zq_tok = mix_logit(logit_of_word<BF16>(sm.raw_q, at), 0.f, false, 0.f, P.invT);
          // the same exponent as the list entries: 2^(z * fp32(log2 e) + c0)
          const double q = (zq_tok >= theta) ? exp2((double)zq_tok * (double)kLog2e + (double)c0) / Zq : 0.0;
          if (q <= 0.0) atomicOr(a.dev_status, MULO_DEV_ZERO_DRAFT_PROB);
          sm.q_tok = q;
        } else {
          atomicOr(a.dev_status, MULO_DEV_DENSE_FALLBACK);
          count_failure(s.reason);
          for (int child = 0; child < rr; ++child)
            defer((size_t)pb * N + t0 + (child / P.r) * P.W + child % P.r);
        }
        learn(0, ok, s.reason, theta, pivot, s.n, n_ge, s.mx);
      }
      q_ok = ok;
    }

    // ------------------------------------------------------------ children
    if (!q_ok) {   // block-uniform: the whole parent went to the general routines
      for (int child = 0; child < rr; ++child) skip_row();
      __syncthreads();   // the predictor written above is read by the next draft row
    } else {
      // where this thread's target entries go: above (below) its own draft entries, up to the first
      // target row of the thread it shares the column with
      const uint32_t t_base = q_base + (uint32_t)(nq * step);
      const uint32_t t_lim = q_lim - (uint32_t)(nq_other * step);
      for (int child = 0; child < rr; ++child) {
        LaneSel& sel = sm.sel[rowi & 1];
        LanePrep& pp = sm.prep[rowi & 1];
        ++rowi;
        const int t = t0 + (child / P.r) * P.W + child % P.r;
        const size_t g = (size_t)pb * N + t;
        float pivot, inv_w, ref;
        choose_pivot(1, std::integral_constant<bool, HAS_U>{}, pivot, inv_w, ref);
        const float c0 = -ref * kLog2e;
        // Two threads prepare the position's uniforms and exp of the logit of x~ (in double).  The
        // logit's words are requested here by asynchronous copies and read after the row has been
        // streamed, so that no warp sits on the load.
        if (tid == kLThreads - 1) {
          const size_t at = g * (size_t)P.V + (size_t)sm.tok[parent & 1];
          cp_async4(&pp.raw_c, logit_word<BF16>(a.cond, at));
          if (HAS_U) cp_async4(&pp.raw_u, logit_word<BF16>(a.uncond, at));
        } else if (tid == kLThreads - 33) {
          const uint4 rnd = philox4x32_10(make_uint4((uint32_t)t, (uint32_t)pb + P.image_offset, P.round, 0u),
                                          make_uint2(P.seed_lo, P.seed_hi));
          pp.rnd[0] = rnd.x;
          pp.rnd[1] = rnd.y;
          pp.rnd[2] = rnd.z;
        }
        uint32_t m_lo, m_hi;
        const int n = stream_row(std::integral_constant<bool, HAS_U>{}, t_base, t_lim, pivot, m_lo, m_hi);
        uint32_t lowm;
        pass_one(sel, t_base, n, pivot, inv_w, c0, lowm);
        if (tid == kLThreads - 1) {
          cp_async_wait_all();
          const size_t at = g * (size_t)P.V + (size_t)sm.tok[parent & 1];
          const float z = mix_logit(logit_of_word<BF16>(pp.raw_c, at), HAS_U ? logit_of_word<BF16>(pp.raw_u, at) : 0.f,
                                    HAS_U, P.cfg_scale, P.invT);
          pp.z_tok = z;
          pp.e_tok = exp2((double)z * (double)kLog2e + (double)c0);   // the list entries' own exponent
        }
        __syncthreads();   // ---- barrier 1
        reset_selection(sm.sel[rowi & 1]);
        Sel s;
        bool ok = locate_bin(sel, s, ref, R - nq - nq_other);
        if (ok) set_aside(sel, t_base, lowm, pivot, inv_w, c0, s.bstar);
        __syncthreads();   // ---- barrier 2
        float theta = 0.f;
        int n_ge = 0;
        double Zp = 1.0;
        if (ok && sel.overflow) {
          ok = false;
          s.reason = 1;
        }
        if (ok) ok = finish_selection(sel, s, theta, n_ge, Zp);
        if (ok && !(Zp > 0.0 && Zp < 1e300)) ok = false;
        if (tid == kLThreads - 1) learn(1, ok, s.reason, theta, pivot, s.n, n_ge, s.mx);
        if (!ok) {   // block-uniform
          if (tid == 0) {
            atomicOr(a.dev_status, MULO_DEV_DENSE_FALLBACK);
            count_failure(s.reason);
            defer(g);
          }
          __syncthreads();   // the predictor
          continue;
        }
        // ---- the decision (Eq. 1 / Eq. 5), the same in every thread
        const double e_tok = (pp.z_tok >= theta) ? pp.e_tok : 0.0;
        const double q_tok = sm.q_tok;
        int accepted;
        if (P.accept_mode == MULO_ACCEPT_THRESHOLD) accepted = e_tok >= P.tau * Zp;
        else if (q_tok <= 0.0) accepted = e_tok > 0.0;
        else accepted = uniform24(pp.rnd[0]) * q_tok * Zp < e_tok;
        const int draws = draws_for(P.resample_mode, accepted);
        const float invZp = (float)(1.0 / Zp);
        if (tid == 0) {
          a.flags[g] = accepted ? 0 : 1;
          if (a.p_tok) a.p_tok[g] = (float)(e_tok / Zp);
          if (a.q_tok) a.q_tok[g] = (float)q_tok;
          if (a.accept_prob) {
            const double p = e_tok / Zp;
            double thr;
            if (P.accept_mode == MULO_ACCEPT_THRESHOLD) thr = p;
            else if (q_tok <= 0.0) thr = p > 0.0 ? 1.0 : 0.0;
            else thr = fmin(1.0, p / q_tok);
            a.accept_prob[g] = (float)thr;
          }
        }

        // ---- the draws.  Weight of an entry (value z, local id = the next set bit of the mask):
        //      residual: max(0, e / Z_p - q) with q from the draft row's list of this thread
        //      (found by popcount on the two masks); target: e.  Entries below theta weigh nothing.
        // One call = the thread's sum, a block scan in double, ONE barrier, and the walk of the
        // thread that owns u * total.  Returns false when the weights have no mass.
        int dcall = 0;   // consecutive draws of a row alternate between the two scan buffers
        auto draw = [&](bool resid, double u, int32_t* out) -> bool {
          auto half_sum = [&](uint32_t m, uint32_t dm, uint32_t ad, int qfirst, float acc) -> float {
            const uint32_t qb = q_base + (uint32_t)(qfirst * step);
            while (m) {
              const uint32_t bit = m & (0u - m);
              m ^= bit;
              const float z = lds_f32(ad);
              ad += step;
              float w = ex2f(fmaf(z, kLog2e, c0));
              if (resid) {
                w = __fmul_rn(w, invZp);
                if (dm & bit) w = fmaxf(__fsub_rn(w, lds_f32(qb + (uint32_t)(__popc(dm & (bit - 1u)) * step))), 0.f);
              }
              if (z >= theta) acc += w;
            }
            return acc;
          };
          const int n_lo = __popc(m_lo), nq_lo = __popc(dm_lo);
          float S = half_sum(m_lo, dm_lo, t_base, 0, 0.f);
          S = half_sum(m_hi, dm_hi, t_base + (uint32_t)(n_lo * step), nq_lo, S);
          // inclusive scan over the warp's threads (ascending ids), warp totals to shared memory
          double inc = (double)S;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const double v = __shfl_up_sync(kFull, inc, o);
            if (lane >= o) inc += v;
          }
          double excl = __shfl_up_sync(kFull, inc, 1);
          if (lane == 0) excl = 0.0;
          double* const wt = sm.w_tot[dcall & 1];
          ++dcall;
          if (lane == 31) wt[warp] = inc;
          __syncthreads();
          double before = 0.0, total = 0.0;
#pragma unroll
          for (int w = 0; w < kLWarps; ++w) {
            const double v = wt[w];
            if (w == warp) before = total;
            total += v;
          }
          if (!(total > 0.0)) return false;
          const double y = u * total;
          const double lo = before + excl, hi = before + inc;
          if (lo <= y && y < hi) {
            // this thread owns u * total: walk its entries with the same arithmetic and order
            int pick = -1, last_pos = -1;
            float acc = 0.f;
            auto half_walk = [&](uint32_t m, uint32_t dm, uint32_t ad, int qfirst, int id0) {
              const uint32_t qb = q_base + (uint32_t)(qfirst * step);
              while (m && pick < 0) {
                const uint32_t bit = m & (0u - m);
                m ^= bit;
                const float z = lds_f32(ad);
                ad += step;
                float w = ex2f(fmaf(z, kLog2e, c0));
                if (resid) {
                  w = __fmul_rn(w, invZp);
                  if (dm & bit) w = fmaxf(__fsub_rn(w, lds_f32(qb + (uint32_t)(__popc(dm & (bit - 1u)) * step))), 0.f);
                }
                if (z >= theta && w > 0.f) {
                  acc += w;
                  last_pos = id0 + __ffs(bit) - 1;
                  if (lo + (double)acc > y) pick = last_pos;
                }
              }
            };
            half_walk(m_lo, dm_lo, t_base, 0, tid * W);
            half_walk(m_hi, dm_hi, t_base + (uint32_t)(n_lo * step), nq_lo, tid * W + 32);
            *out = pick >= 0 ? pick : last_pos;   // rounding left the sum short: the last id with weight
          }
          return true;
        };
        if (draws & kDrawResidual) {
          const double u1 = uniform24(pp.rnd[1]);
          if (!draw(true, u1, a.cand_res + g)) draw(false, u1, a.cand_res + g);   // a residual without mass
        }
        if (draws & kDrawTarget) draw(false, uniform24(pp.rnd[2]), a.cand_tgt + g);
      }
    }
  }
#undef rslot
#undef rphase
}

}  // namespace mulo
