// The fast path of the fused round for rows with top-k on, when the vocabulary splits
// evenly over a CTA's 256 threads (V = 256 * W, W <= 64 ids per thread).
//
// A persistent CTA (256 threads, three per SM) owns a contiguous range of parent (low-res)
// cells.  Per parent it streams the draft row and then its r*r target rows ONCE.  Every WARP has
// a two-slot shared-memory ring of its own: a slot holds one PHASE of the warp's part of a row,
// brought by a tiled bulk-tensor copy (never multicast) -- 32 bytes for every lane, the next
// 16 bf16 (8 fp32) ids of the 64-id range that thread owns, of the conditional and of the
// unconditional row, placed with the 32-byte swizzle so that the 128-bit shared loads of a
// quarter warp hit eight different bank groups.  A warp waits for its own data only and requests
// its next phase itself, the moment the slot's words are in registers; the warps of a CTA meet
// at the row's first block barrier.  Owning a CONTIGUOUS id range is what keeps the rest cheap:
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
constexpr int kLTile = 32 * 32;          // bytes of one tensor's tile of one warp: 32 bytes per lane
constexpr int kLSlot = 2 * kLTile;       // conditional + unconditional
constexpr int kLWarpRing = kLStages * kLSlot;   // ring bytes of one warp
constexpr int kLRing = kLWarps * kLWarpRing;    // ring bytes of the CTA
constexpr int kLBins = 256;
constexpr int kLSetAside = 64;           // entries of the crossing bin that are ranked exactly
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNearRefGap = 8.0f;      // a row whose maximum lies further from the predicted exp reference is summed
                                         // again against its own maximum (large exponents cost relative accuracy)
constexpr float kMaxRefGap = 60.0f;      // ... and beyond this the first sum may have left fp32's range: the row is given up

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
  int age;                    // rows learnt from since the prediction was last lost
  float theta, rho, mx;       // running k-th largest, density below it, row maximum
  float pivot, inv_w, ref;    // what the next row starts from (valid while have != 0)
  float shift, step;          // bootstrap adaptation, as in the general streaming kernel
  int dir;
};

constexpr int kLMaxRows = 17;  // draft row + r*r children, r <= 4

// Selection scratch of one row.  Two copies, used by rows of alternating parity: what a row adds
// into (histogram, set-aside list, per-warp partials) is reset / rewritten two rows later, with
// at least two block barriers in between, so no reader of row i can meet a writer of row i + 2.
struct LaneSel {
  alignas(16) unsigned hist[kLBins];
  float sa_z[kLSetAside];
  float sa_e[kLSetAside];
  unsigned short sa_owner[kLSetAside];   // the thread whose list holds the entry
  unsigned n_sa;
  unsigned overflow;
  unsigned n_total;            // candidates of the row (integer atomics: order-free)
  unsigned max_key;            // order-preserving key of the row maximum
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
  uint64_t full[kLWarps][kLStages];   // every warp has a ring of its own
  LaneSel sel[2];
  LanePrep prep[2];
  double w_tot[2][kLWarps];    // block scan of a draw; consecutive draws alternate
  float red[kLWarps][2];
  unsigned char cnt[kLThreads];
  LanePredictor pred[2];
  double q_tok;                // of the current parent
  uint32_t raw_q;              // landing place of the draft logit word of x~
  int tok[2];                  // the draft token of the parent in work / of the next one
  int rows[2][kLMaxRows];      // row index (within its tensor) of every row of a parent, by parent parity
  int image[2];                // image index of the parent, by parent parity
  int abort;                   // a wait of this CTA gave up: stop at the next row's first barrier
};

__device__ __forceinline__ void tma_tile_3d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"((uint64_t)tm), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(bar))
      : "memory");
}
// Bounded wait on a ring slot: after kSpinLimit tries the wait gives up, raises the time-out bit
// and the CTA's abort flag; once that flag is up every later wait of the CTA returns at once, and
// the CTA stops at the next row's first barrier.
__device__ __forceinline__ void lane_wait(uint64_t* bar, uint32_t parity, uint32_t* dev_status, volatile int* abort) {
  if (mbar_try_wait(bar, parity)) return;
  if (*abort) return;
#pragma unroll 1
  for (uint32_t it = 0; it < kSpinLimit; ++it)
    if (mbar_try_wait(bar, parity)) return;
  atomicOr(dev_status, MULO_DEV_TIMEOUT);
  *abort = 1;
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

// Appends z to a thread's list if z >= pivot: four instructions -- compare, store, cursor step,
// the survivor's bit in the mask -- the last three predicated.  Written in PTX: left to the
// compiler, the same statements become a branch and several moves per element.  `stp` is the
// thread's step (+-512 bytes, or 0 once its column has no room left for a whole phase).
template <int BIT>
__device__ __forceinline__ void lane_put(float z, float pivot, uint32_t& cur, uint32_t stp, uint32_t& m) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ge.f32 p, %2, %3;\n\t"
      "@p st.shared.f32 [%0], %2;\n\t"
      "@p add.u32 %0, %0, %4;\n\t"
      "@p or.b32 %1, %1, %5;\n\t}"
      : "+r"(cur), "+r"(m)
      : "f"(z), "f"(pivot), "r"(stp), "n"(1u << BIT)
      : "memory");
}

template <int J>
__device__ __forceinline__ uint32_t word_of(const uint4& v) {
  return J == 0 ? v.x : J == 1 ? v.y : J == 2 ? v.z : v.w;
}

// Two ids of a phase: word J of 16-byte piece I of the thread's 32 bytes.  bf16: one word of the
// conditional (and unconditional) row holds both; fp32: words 2J and 2J + 1 of piece I hold them
// (J < 2).  Pre-processing as the definition says (d = c - u; v = fma(s, d, u); z = v * invT, each
// one fp32 rounding; two ids per packed instruction), then the two appends.
template <bool BF16, bool ROW_U, bool SCALE, int I, int J>
__device__ __forceinline__ void lane_pair(const uint4 (&c)[2], const uint4 (&u)[2], float2 s2, float2 t2,
                                          float pivot, uint32_t& cur, uint32_t stp, uint32_t& m) {
  float2 v, un;
  if (BF16) {
    const uint32_t cw = word_of<J>(c[I]);
    v = make_float2(bf16_lo(cw), bf16_hi(cw));
    if (ROW_U) {
      const uint32_t uw = word_of<J>(u[I]);
      un = make_float2(bf16_lo(uw), bf16_hi(uw));
    }
  } else {
    v = make_float2(__uint_as_float(word_of<(2 * J) & 3>(c[I])), __uint_as_float(word_of<(2 * J + 1) & 3>(c[I])));
    if (ROW_U)
      un = make_float2(__uint_as_float(word_of<(2 * J) & 3>(u[I])), __uint_as_float(word_of<(2 * J + 1) & 3>(u[I])));
  }
  if (ROW_U) v = __ffma2_rn(s2, __ffma2_rn(un, make_float2(-1.f, -1.f), v), un);   // fma(u, -1, c) rounds as c - u
  if (SCALE) v = __fmul2_rn(v, t2);
  constexpr int bit = BF16 ? I * 8 + J * 2 : I * 4 + J * 2;
  lane_put<bit>(v.x, pivot, cur, stp, m);
  lane_put<bit + 1>(v.y, pivot, cur, stp, m);
}

// One phase of a row for one thread, in two steps.  lane_load: the 32 bytes (16 bf16 / 8 fp32 ids)
// of the conditional row at `sb` and of the unconditional row one tile further, into registers
// (after which the slot can be refilled).  lane_dense: survivors z >= pivot are appended at `cur`
// (stepping by STEP bytes, clamped at `lim`) and marked in the returned mask.
template <bool ROW_U>
__device__ __forceinline__ void lane_load(uint32_t sb, uint32_t sw, uint4 (&c)[2], uint4 (&u)[2]) {
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    c[i] = lds128(sb + (((uint32_t)i ^ sw) << 4));
    u[i] = ROW_U ? lds128(sb + kLTile + (((uint32_t)i ^ sw) << 4)) : make_uint4(0, 0, 0, 0);
  }
}
template <bool BF16, bool ROW_U, bool SCALE>
__device__ __forceinline__ uint32_t lane_dense(const uint4 (&c)[2], const uint4 (&u)[2], float s, float invT,
                                               float pivot, uint32_t& cur, uint32_t stp) {
  const float2 s2 = make_float2(s, s), t2 = make_float2(invT, invT);
  uint32_t m = 0;
  lane_pair<BF16, ROW_U, SCALE, 0, 0>(c, u, s2, t2, pivot, cur, stp, m);
  lane_pair<BF16, ROW_U, SCALE, 0, 1>(c, u, s2, t2, pivot, cur, stp, m);
  if (BF16) {
    lane_pair<BF16, ROW_U, SCALE, 0, 2>(c, u, s2, t2, pivot, cur, stp, m);
    lane_pair<BF16, ROW_U, SCALE, 0, 3>(c, u, s2, t2, pivot, cur, stp, m);
  }
  lane_pair<BF16, ROW_U, SCALE, 1, 0>(c, u, s2, t2, pivot, cur, stp, m);
  lane_pair<BF16, ROW_U, SCALE, 1, 1>(c, u, s2, t2, pivot, cur, stp, m);
  if (BF16) {
    lane_pair<BF16, ROW_U, SCALE, 1, 2>(c, u, s2, t2, pivot, cur, stp, m);
    lane_pair<BF16, ROW_U, SCALE, 1, 3>(c, u, s2, t2, pivot, cur, stp, m);
  }
  return m;
}

// 2^x in double, out of line: three call sites, a few hundred instructions each otherwise
__device__ __noinline__ double lane_exp2(double x) { return exp2(x); }

// Philox4x32-10 as a rolled loop (one thread per row runs it; the unrolled form is ten times the code)
__device__ __noinline__ uint4 lane_philox(uint4 c, uint2 k) {
#pragma unroll 1
  for (int i = 0; i < 10; ++i) {
    const uint32_t a = 0xD2511F53u, b = 0xCD9E8D57u;
    const uint32_t h0 = __umulhi(a, c.x), l0 = a * c.x;
    const uint32_t h1 = __umulhi(b, c.z), l1 = b * c.z;
    c = make_uint4(h1 ^ c.y ^ k.x, l1, h0 ^ c.w ^ k.y, l0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}

// The optional probability outputs of a position (one thread; out of line: double divisions).
__device__ __noinline__ void lane_write_probs(float* p_tok, float* q_tok_out, float* accept_prob, size_t g, double e_tok,
                                              double q_tok, double Z, bool threshold_rule) {
  const double p = e_tok / Z;
  if (p_tok) p_tok[g] = (float)p;
  if (q_tok_out) q_tok_out[g] = (float)q_tok;
  if (accept_prob) {
    double thr;
    if (threshold_rule) thr = p;
    else if (q_tok <= 0.0) thr = p > 0.0 ? 1.0 : 0.0;
    else thr = fmin(1.0, p / q_tok);
    accept_prob[g] = (float)thr;
  }
}

// The predictor of one kind of row after a row (ok: theta found exactly).  One thread; out of line.
__device__ __noinline__ void lane_learn(LanePredictor* prp, bool ok, int reason, float theta, float pivot, int n,
                                        int n_ge, float mx, int margin, float a_theta, float a_boot) {
  LanePredictor pr = *prp;
  if (!ok) {
    pr.have = 0;
    pr.age = 0;
    const int dir = reason == 2 ? -1 : (reason == 1 || reason == 3) ? 1 : 0;
    if (dir != 0) {
      const float unit = 0.5f * (a_theta - a_boot);
      if (pr.dir == 0) pr.step = unit;
      else if (pr.dir == dir) pr.step = fminf(2.0f * pr.step, 64.0f * unit);
      else pr.step = fmaxf(0.5f * pr.step, 0.25f * unit);
      pr.shift += (float)dir * pr.step;
      pr.dir = dir;
    }
  } else {
    pr.dir = 0;
    const int below = n - n_ge;   // candidates in [pivot, theta)
    // running means: a plain average over the first four rows, weight 1/4 for the newest after that
    const float w_new = pr.have ? fmaxf(0.25f, 1.0f / (float)(pr.age + 1)) : 1.0f;
    float rho = pr.rho;
    bool rho_ok = pr.have != 0;
    if (theta > pivot && below >= 16) {
      const float r_new = (float)below / (theta - pivot);
      rho = pr.have ? pr.rho + w_new * (r_new - pr.rho) : r_new;
      rho_ok = true;
    }
    if (!rho_ok) {
      pr.have = 0;
      pr.age = 0;
    } else {
      pr.theta = pr.have ? pr.theta + w_new * (theta - pr.theta) : theta;
      pr.mx = pr.have ? pr.mx + w_new * (mx - pr.mx) : mx;
      pr.rho = rho;
      pr.have = 1;
      if (pr.age < 8) ++pr.age;
      // a prediction that rests on a single row carries that row's noise in the threshold and in
      // the density: the row after it aims for a wider margin
      const float d = (pr.age < 2 ? 1.4f : 1.0f) * (float)margin / rho;
      pr.pivot = pr.theta - d;
      pr.inv_w = (float)kLBins / (2.0f * d);   // the histogram spans twice the distance pivot -> threshold
      pr.ref = pr.mx;
    }
  }
  *prp = pr;
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
  // A list column (R rows of 512 bytes; lane l of a warp sits in bank l) holds four stacks: the
  // draft row's entries of thread c from row 0 upwards and of c + 128 from row R - 1 downwards (fixed
  // while the parent's children are verified), and between them the current target row's entries
  // of two OTHER threads, c ^ 64 and (c ^ 64) + 128, again growing towards each other.  (A thread's
  // draft and target entries cover the same ids and their counts rise and fall together, the target
  // rows being the draft row plus noise: four stacks of four different id ranges overflow far more
  // rarely than two pairs.)  A stack is clamped at the first row of the stack it grows towards, so
  // it can never reach the draft entries at the column's other end; whether the two target stacks
  // met is checked from the four counts.
  const bool up = tid < kLThreads / 2;
  const int step = up ? 512 : -512;
  const int colq = tid & 127, colt = colq ^ 64;   // the columns of this thread's draft / target stack
  const uint32_t col = ring + kLRing + (uint32_t)colq * 4u;
  const uint32_t tcol = ring + kLRing + (uint32_t)colt * 4u;
  const uint32_t q_base = col + (up ? 0u : (uint32_t)(R - 1) * 512u);
  const uint32_t q_lim = col + (up ? (uint32_t)(R - 1) * 512u : 0u);   // the partner's first draft row
  const uint32_t sw = ((uint32_t)lane >> 2) & 1u;          // 32-byte swizzle: address bit 4 ^= bit 7
  const uint32_t wring = ring + (uint32_t)warp * kLWarpRing;   // this warp's ring
  const uint32_t my_off = (uint32_t)lane * 32u;

  if (tid == 0) {
    for (int w = 0; w < kLWarps; ++w)
      for (int s = 0; s < kLStages; ++s) mbar_init(&sm.full[w][s], 1);
    mbar_fence_init();
    sm.abort = 0;
    for (int s = 0; s < 2; ++s) {
      sm.sel[s].n_sa = 0;
      sm.sel[s].overflow = 0;
      sm.sel[s].n_total = 0;
      sm.sel[s].max_key = 0;
      LanePredictor& pr = sm.pred[s];
      pr.have = 0;
      pr.age = 0;
      pr.theta = 0.f; pr.rho = 1.f; pr.mx = 0.f;
      pr.pivot = 0.f; pr.inv_w = 0.f; pr.ref = 0.f;
      pr.shift = 0.f; pr.step = 0.f; pr.dir = 0;
    }
  }
  sm.sel[0].hist[tid] = 0;
  sm.sel[1].hist[tid] = 0;
  __syncthreads();

  // ---- the rings: a warp's items (the phases of its rows) in the order it consumes them; lane 0
  //      requests item n + kLStages into the slot of item n as soon as the warp has read it
  // row indices of a parent's rows, for the warps' requests (one thread; slot = parity of the parent)
  auto fill_rows = [&](int parent) {
    const int hw = P.h * P.w;
    const int b = parent / hw, rem = parent - b * hw, ca = rem / P.w, cc = rem - ca * P.w;
    int* rows = sm.rows[parent & 1];
    sm.image[parent & 1] = b;
    rows[0] = parent;
    int j = 1;
    for (int di = 0; di < P.r; ++di)
      for (int dj = 0; dj < P.r; ++dj, ++j) rows[j] = b * N + (ca * P.r + di) * P.W + cc * P.r + dj;
  };
  // The next item this warp requests: phase c_ph of row c_j of parent c_par, c_left items to go (the
  // same in all its lanes; stepping it is a few uniform instructions, the requests are lane 0's).
  int c_ph = 0, c_j = 0, c_par = p_begin, c_left = (p_end - p_begin) * rows_per_parent * n_ph;
  auto cursor_issue = [&](int slot) {
    if (lane == 0) {
      const uint32_t dst = wring + (uint32_t)slot * kLSlot;
      uint64_t* bar = &sm.full[warp][slot];
      const int row = sm.rows[c_par & 1][c_j];
      if (c_j == 0) {
        mbar_expect_tx(bar, kLTile);
        tma_tile_3d(dst, &tm_q, IDS * c_ph, 32 * warp, row, bar);
      } else {
        mbar_expect_tx(bar, HAS_U ? kLSlot : kLTile);
        tma_tile_3d(dst, &tm_c, IDS * c_ph, 32 * warp, row, bar);
        if (HAS_U) tma_tile_3d(dst + kLTile, &tm_u, IDS * c_ph, 32 * warp, row, bar);
      }
    }
    --c_left;
    if (++c_ph == n_ph) {
      c_ph = 0;
      if (++c_j == rows_per_parent) {
        c_j = 0;
        ++c_par;
      }
    }
  };
  if (tid == 0) {
    fill_rows(p_begin);
    if (p_begin + 1 < p_end) fill_rows(p_begin + 1);
  }
  __syncthreads();
  for (int s = 0; s < kLStages; ++s)
    if (c_left > 0) cursor_issue(s);
  int rs = 0;   // slots consumed so far: bit 0 = the slot to read next, bit 1 = its phase
#define rslot (rs & 1)
#define rphase ((uint32_t)(rs >> 1) & 1u)
  static_assert(kLStages == 2, "the packed ring state assumes two slots");
  // The warp has the slot's words in registers: request the next item into it.  The lanes of a
  // warp may drift apart wherever one of them does something alone (the requests below, the
  // bookkeeping of a failed row); they meet here, before the request -- so that no lane still has
  // the slot to read -- and after it -- so that none runs on to wait for an item that lane 0 has
  // not requested yet, or falls a whole barrier phase behind.  (`loaded` is one of the slot's
  // words: naming it keeps the loads before the meeting point.)
  auto release_slot = [&](uint32_t loaded) {
    asm volatile("" ::"r"(loaded) : "memory");
    __syncwarp();
    if (c_left > 0) cursor_issue(rslot);
    __syncwarp();
    ++rs;
  };
  auto skip_row = [&]() {
    for (int ph = 0; ph < n_ph; ++ph) {
      lane_wait(&sm.full[warp][rslot], rphase, a.dev_status, &sm.abort);
      release_slot(0u);
    }
  };

  // ---- pivot, histogram scale and exp reference of the next row of a kind
  auto choose_pivot = [&](int kind, const bool row_u, float& pivot, float& inv_w, float& ref) {
    if (sm.pred[kind].have) {   // block-uniform
      pivot = sm.pred[kind].pivot;
      inv_w = sm.pred[kind].inv_w;
      ref = sm.pred[kind].ref;
      return;
    }
    const LanePredictor pr = sm.pred[kind];
    // no prediction: mean and spread of the row's first phase (every thread's first ids: an
    // even sample of the row), assuming a normal shape; the slot is read again by the dense pass
    lane_wait(&sm.full[warp][rslot], rphase, a.dev_status, &sm.abort);
    const uint32_t sb = wring + (uint32_t)rslot * kLSlot + my_off;
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const uint4 c = lds128(sb + (((uint32_t)i ^ sw) << 4));
      uint4 u = make_uint4(0, 0, 0, 0);
      if (row_u) u = lds128(sb + kLTile + (((uint32_t)i ^ sw) << 4));
      const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, uw[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (BF16) {
          const float z0 = mix_logit(bf16_lo(cw[j]), bf16_lo(uw[j]), row_u, P.cfg_scale, P.invT);
          const float z1 = mix_logit(bf16_hi(cw[j]), bf16_hi(uw[j]), row_u, P.cfg_scale, P.invT);
          s1 += z0 + z1;
          s2 += z0 * z0 + z1 * z1;
        } else {
          const float z0 = mix_logit(__uint_as_float(cw[j]), __uint_as_float(uw[j]), row_u, P.cfg_scale, P.invT);
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
    inv_w = (float)kLBins / (3.0f * d);   // (a predicted row's histogram spans 2 d)
    ref = mean + a.a_max * sd;
  };

  // ---- a row through the ring into this thread's list (from `base` towards `lim`, the first row of
  //      the stack it grows towards); returns the entry count.  Before a phase the thread makes sure
  //      that a whole phase's worth of rows is left; if not, its cursor stops (the appends of the
  //      rest of the row land on one row) and the row is given up after the next barrier.
  auto stream_row = [&](LaneSel& sel, const bool row_u, uint32_t base, uint32_t lim, float pivot, uint32_t& m_lo,
                        uint32_t& m_hi) -> int {
    uint32_t cur = base;
    m_lo = 0;
    m_hi = 0;
#pragma unroll 1
    for (int ph = 0; ph < n_ph; ++ph) {
      lane_wait(&sm.full[warp][rslot], rphase, a.dev_status, &sm.abort);
      const uint32_t room = (up ? lim - cur : cur - lim) >> 9;   // rows between the cursor and the other stack
      uint32_t stp = (uint32_t)step;
      if (room < (uint32_t)IDS) {
        stp = 0u;
        sel.overflow = 1;
      }
      uint4 c[2], u[2];
      uint32_t m;
      const uint32_t sb = wring + (uint32_t)rslot * kLSlot + my_off;
      // (the variants differ in compile-time constants only; the branches are block-uniform)
      if (HAS_U && row_u) {
        lane_load<true>(sb, sw, c, u);
        release_slot(c[1].w ^ u[1].w);
        m = scale ? lane_dense<BF16, true, true>(c, u, P.cfg_scale, P.invT, pivot, cur, stp)
                  : lane_dense<BF16, true, false>(c, u, P.cfg_scale, P.invT, pivot, cur, stp);
      } else {
        lane_load<false>(sb, sw, c, u);
        release_slot(c[1].w);
        m = scale ? lane_dense<BF16, false, true>(c, u, P.cfg_scale, P.invT, pivot, cur, stp)
                  : lane_dense<BF16, false, false>(c, u, P.cfg_scale, P.invT, pivot, cur, stp);
      }
      const int bit0 = ph * IDS;
      if (bit0 < 32) m_lo |= m << bit0;
      else m_hi |= m << (bit0 - 32);
    }
    return (int)((up ? cur - base : base - cur) >> 9);
  };

  // ---- pass 1 over the thread's own entries: exp against the reference, maximum, histogram of
  //      the low end; per-warp partial results for the block
  auto pass_one = [&](LaneSel& sel, uint32_t base, int n, float pivot, float inv_w, float c0, uint32_t& lowm) -> float {
    const float hoff = -pivot * inv_w;
    float mx = -INFINITY, s_all = 0.f;
    lowm = 0;
    // four entries per trip, every warp lane making the same number of trips (a lane past its own
    // end loads nothing and works on -inf: no weight, no bin), so that the four chains of
    // load -> exp -> add overlap and the loop needs no divergence handling
    const int nmax = __reduce_max_sync(kFull, n);
    uint32_t ad = base;
    for (int i0 = 0; i0 < nmax; i0 += 4, ad += 4 * step) {
      float z[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) z[k] = i0 + k < n ? lds_f32(ad + (uint32_t)(k * step)) : -INFINITY;
      uint32_t low4 = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        mx = fmaxf(mx, z[k]);
        s_all += ex2f(fmaf(z[k], kLog2e, c0));
        // (a column whose stacks have met holds entries from below the pivot until the row is
        // given up after the next barrier: the unsigned compare keeps their bins out of range)
        const unsigned bin = (unsigned)(int)fmaf(z[k], inv_w, hoff);
        if (bin < (unsigned)kLBins) {
          atomicAdd(&sel.hist[bin], 1u);
          low4 |= 1u << k;
        }
      }
      lowm |= low4 << (i0 & 31);
    }
    sm.cnt[tid] = (unsigned char)n;
    const int nsum = __reduce_add_sync(kFull, n);
    const unsigned mk = __reduce_max_sync(kFull, float_key(mx));
    const double es = warp_sum((double)s_all);
    if (lane == 0) {
      atomicAdd(&sel.n_total, (unsigned)nsum);
      atomicMax(&sel.max_key, mk);
      sel.w_e[warp] = es;
    }
    return s_all;   // exp of ALL of this thread's entries, in list order
  };

  // a row whose maximum turned out far from the predicted reference: the sum once more, against
  // the maximum itself (between the row's first and second barrier)
  auto sum_again = [&](LaneSel& sel, uint32_t base, int n, float c0) -> float {
    float s_all = 0.f;
    uint32_t ad = base;
#pragma unroll 1
    for (int i = 0; i < n; ++i, ad += step) s_all += ex2f(fmaf(lds_f32(ad), kLog2e, c0));
    const double es = warp_sum((double)s_all);
    if (lane == 0) sel.w_e[warp] = es;
    return s_all;
  };

  struct Sel {
    int n, bstar, want, cum, reason;
    float mx;
  };
  // after the barrier that follows pass_one (every warp computes the same)
  auto locate_bin = [&](LaneSel& sel, Sel& s, float ref, int rows) -> bool {
    const int n = (int)sel.n_total;
    const float mx = key_float(sel.max_key);
    s.n = n;
    s.mx = mx;
    s.reason = 0;
    // the two stacks that grow towards each other must fit the `rows` they share; the bit mask of a
    // thread's low entries covers 32 entries
    const int mine_n = sm.cnt[tid], other_n = sm.cnt[tid ^ 128];
    if (__any_sync(kFull, mine_n + other_n > rows || mine_n > 32) && lane == 0) sel.overflow = 1;
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
    static_assert(PER == 8, "a lane reads its eight bins with two 128-bit loads");
    unsigned h[PER];
    {
      const uint4 h0 = *reinterpret_cast<const uint4*>(&sel.hist[lane * PER]);
      const uint4 h1 = *reinterpret_cast<const uint4*>(&sel.hist[lane * PER + 4]);
      h[0] = h0.x; h[1] = h0.y; h[2] = h0.z; h[3] = h0.w;
      h[4] = h1.x; h[5] = h1.y; h[6] = h1.z; h[7] = h1.w;
    }
    unsigned mine = 0;
#pragma unroll
    for (int b = 0; b < PER; ++b) mine += h[b];
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
  auto set_aside = [&](LaneSel& sel, uint32_t base, uint32_t lowm, float pivot, float inv_w, float c0, int bstar) -> float {
    const float hoff = -pivot * inv_w;
    float excl = 0.f;
    // four low entries per trip (their loads and bins overlap); a thread has two or three on average
    const int trips = (__reduce_max_sync(kFull, __popc(lowm)) + 3) >> 2;
    for (int it = 0; it < trips; ++it) {
      float z[4];
      int bin[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int i = __ffs(lowm) - 1;   // -1: none left
        lowm &= lowm - 1;
        z[k] = i >= 0 ? lds_f32(base + (uint32_t)(i * step)) : INFINITY;
        bin[k] = (int)fmaf(z[k], inv_w, hoff);   // +inf -> a bin above every other
      }
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (bin[k] <= bstar) {
          const float e = ex2f(fmaf(z[k], kLog2e, c0));
          if (bin[k] < bstar) excl += e;
          else {
            const unsigned at = atomicAdd(&sel.n_sa, 1u);
            if (at < (unsigned)kLSetAside) {
              sel.sa_z[at] = z[k];
              sel.sa_e[at] = e;
              sel.sa_owner[at] = (unsigned short)tid;
            }
          }
        }
    }
    const double ex = warp_sum((double)excl);
    if (lane == 0) sel.w_excl[warp] = ex;
    return excl;   // exp of this thread's entries below the crossing bin
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
    // the eight warps' partial sums: one per lane, added in a fixed butterfly order
    double z = lane < kLWarps ? sel.w_e[lane] - sel.w_excl[lane] : 0.0;
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) z += __shfl_xor_sync(kFull, z, o);
    z = __shfl_sync(kFull, z, 0);
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
      sel.n_total = 0;
      sel.max_key = 0;
    }
  };

  uint32_t dm_lo = 0, dm_hi = 0;   // survivor mask of the parent's draft row (this thread's ids)
  int nq = 0;                      // draft entries of this thread
  int nq_up = 0, nq_dn = 0;        // draft entries at the two ends of the column that takes its target entries
  int rowi = 0;                    // rows done by this CTA (its parity selects the scratch copies)

  if (tid == kLThreads - 1) sm.tok[p_begin & 1] = __ldg(a.draft_tok_lo + p_begin);
  for (int parent = p_begin; parent < p_end; ++parent) {
    const int pb = sm.image[parent & 1];   // (tables written at least two barriers ago)
    // One loop body for the draft row (j = 0) and the r*r target rows under it: the two kinds of row
    // share every pass up to the exact threshold, and one copy of the code is what the
    // instruction cache holds.
#pragma unroll 1
    for (int j = 0; j <= rr; ++j) {
      const bool is_q = j == 0;
      LaneSel& sel = sm.sel[rowi & 1];
      LanePrep& pp = sm.prep[rowi & 1];
      ++rowi;
      const size_t g = (size_t)sm.rows[parent & 1][j];   // a target row's position b * N + t (the draft row's cell)
      const int t = (int)g - pb * N;
      // a draft row's entries go where other threads kept the previous parent's target entries: the
      // thread that walked the last draw must be done with them
      if (is_q && parent > p_begin) __syncthreads();
      float pivot, inv_w, ref;
      choose_pivot(is_q ? 0 : 1, HAS_U && !is_q, pivot, inv_w, ref);
      float c0 = -ref * kLog2e;
      // Two threads prepare what the row needs besides its lists: the logit of x~ (requested here by
      // asynchronous copies, read after the row has been streamed, so that no warp sits on the load)
      // and the position's uniforms.
      if (tid == kLThreads - 1) {
        if (is_q) {
          cp_async_wait_all();   // the token, requested a parent ago
          const int tok = checked_token(sm.tok[parent & 1], P.V, a.dev_status);
          sm.tok[parent & 1] = tok;
          cp_async4(&sm.raw_q, logit_word<BF16>(a.draft, (size_t)parent * P.V + (size_t)tok));
          if (parent + 1 < p_end) cp_async4(&sm.tok[(parent + 1) & 1], a.draft_tok_lo + parent + 1);
        } else {
          const size_t at = g * (size_t)P.V + (size_t)sm.tok[parent & 1];
          cp_async4(&pp.raw_c, logit_word<BF16>(a.cond, at));
          if (HAS_U) cp_async4(&pp.raw_u, logit_word<BF16>(a.uncond, at));
        }
      } else if (tid == kLThreads - 33 && !is_q) {
        const uint4 rnd = lane_philox(make_uint4((uint32_t)t, (uint32_t)pb + P.image_offset, P.round, 0u),
                                      make_uint2(P.seed_lo, P.seed_hi));
        pp.rnd[0] = rnd.x;
        pp.rnd[1] = rnd.y;
        pp.rnd[2] = rnd.z;
      }
      // where the row's entries go: the draft row's from the end of the column, a target row's from
      // the end of the thread's draft entries, up to the first target row of the other thread
      const uint32_t t_first = tcol + (uint32_t)nq_up * 512u, t_last = tcol + (uint32_t)(R - 1 - nq_dn) * 512u;
      const uint32_t base = is_q ? q_base : up ? t_first : t_last;
      const uint32_t lim = is_q ? q_lim : up ? t_last : t_first;
      uint32_t m_lo, m_hi;
      const int n = stream_row(sel, HAS_U && !is_q, base, lim, pivot, m_lo, m_hi);
      uint32_t lowm;
      const float s_all = pass_one(sel, base, n, pivot, inv_w, c0, lowm);
      if (tid == kLThreads - 1 && !is_q) {
        cp_async_wait_all();
        const size_t at = g * (size_t)P.V + (size_t)sm.tok[parent & 1];
        const float z = mix_logit(logit_of_word<BF16>(pp.raw_c, at), HAS_U ? logit_of_word<BF16>(pp.raw_u, at) : 0.f,
                                  HAS_U, P.cfg_scale, P.invT);
        pp.z_tok = z;
        pp.e_tok = lane_exp2((double)z * (double)kLog2e + (double)c0);   // the list entries' own exponent
      }
      __syncthreads();   // ---- barrier 1
      if (*(volatile int*)&sm.abort) {   // block-uniform: the flag was raised before the barrier
        // Nothing more is written for this CTA's rows (the status bit says that the call's results
        // are invalid).  Before its shared memory is given up, every warp waits -- bounded again --
        // for the copies it still has in flight: the items it requested and did not consume.
        const int issued = (p_end - p_begin) * rows_per_parent * n_ph - c_left;
        for (; rs < issued; ++rs)
          for (uint32_t it = 0; it < (1u << 16); ++it)
            if (mbar_try_wait(&sm.full[warp][rslot], rphase)) break;
        return;
      }
      reset_selection(sm.sel[rowi & 1]);
      Sel s;
      bool ok = locate_bin(sel, s, ref, is_q ? R : R - nq_up - nq_dn);
      if (is_q) {
        nq_up = sm.cnt[colt];
        nq_dn = sm.cnt[colt + 128];
        // the warps are requesting rows of this parent and (at its end) of the next; the table entry of
        // the parent after that replaces the previous parent's, whose last request is behind every warp
        if (tid == 64 && parent + 1 < p_end && parent > p_begin) fill_rows(parent + 1);
      }
      float s_inc = s_all;   // becomes: exp of this thread's entries that are >= theta
      if (ok && !(fabsf(s.mx - ref) <= kNearRefGap)) {   // block-uniform, rare
        c0 = -s.mx * kLog2e;
        s_inc = sum_again(sel, base, n, c0);
        if (tid == kLThreads - 1 && !is_q) pp.e_tok = lane_exp2((double)pp.z_tok * (double)kLog2e + (double)c0);
      }
      if (ok) s_inc -= set_aside(sel, base, lowm, pivot, inv_w, c0, s.bstar);
      __syncthreads();   // ---- barrier 2
      float theta = 0.f;
      int n_ge = 0;
      double Z = 1.0;
      if (ok && sel.overflow) {
        ok = false;
        s.reason = 1;
      }
      if (ok) ok = finish_selection(sel, s, theta, n_ge, Z);
      if (ok && !(Z > 0.0 && Z < 1e300)) ok = false;
      if (tid == kLThreads - 1)
        lane_learn(&sm.pred[is_q ? 0 : 1], ok, s.reason, theta, pivot, s.n, n_ge, s.mx, a.margin, a.a_theta, a.a_boot);

      if (is_q) {
        // ------------------------------------------------------------ the draft row ends here
        if (!ok) {   // block-uniform: the whole parent goes to the general routines
          if (tid == 0) {
            atomicOr(a.dev_status, MULO_DEV_DENSE_FALLBACK);
            count_failure(s.reason);
            for (int ch = 1; ch <= rr; ++ch) defer((size_t)sm.rows[parent & 1][ch]);
          }
          for (int ch = 0; ch < rr; ++ch) skip_row();
          __syncthreads();   // the predictor written above is read by the next draft row
          break;
        }
        dm_lo = m_lo;
        dm_hi = m_hi;
        nq = n;
        {   // q in place of z: q(x) = [z >= theta] exp(z - ref) / Z_q, the fp32 product of e and 1/Z_q
          const float invZq = 1.0f / (float)Z;
          uint32_t ad = q_base;
#pragma unroll 2
          for (int i = 0; i < nq; ++i, ad += step) {
            const float z = lds_f32(ad);
            const float e = ex2f(fmaf(z, kLog2e, c0));
            sts_f32(ad, z >= theta ? __fmul_rn(e, invZq) : 0.f);
          }
        }
        if (tid == kLThreads - 1) {
          cp_async_wait_all();
          const size_t at = (size_t)parent * P.V + (size_t)sm.tok[parent & 1];
          const float zq_tok = mix_logit(logit_of_word<BF16>(sm.raw_q, at), 0.f, false, 0.f, P.invT);
          // the same exponent as the list entries: 2^(z * fp32(log2 e) + c0)
          const double q = (zq_tok >= theta) ? lane_exp2((double)zq_tok * (double)kLog2e + (double)c0) / Z : 0.0;
          if (q <= 0.0) atomicOr(a.dev_status, MULO_DEV_ZERO_DRAFT_PROB);
          sm.q_tok = q;
        }
        continue;
      }

      // ------------------------------------------------------------ a target row goes on
      if (!ok) {   // block-uniform
        if (tid == 0) {
          atomicOr(a.dev_status, MULO_DEV_DENSE_FALLBACK);
          count_failure(s.reason);
          defer(g);
        }
        __syncthreads();   // the predictor
        continue;
      }
      {   // this thread's entries of the crossing bin that fell below theta (their slots were handed
          // out in no fixed order: summed in double, which is exact for values of one bin, the
          // result does not depend on it)
        const int mcount = (int)sel.n_sa;
        double mine = 0.0;
        for (int i = 0; i < mcount; ++i)
          if (sel.sa_owner[i] == tid && sel.sa_z[i] < theta) mine += (double)sel.sa_e[i];
        s_inc = fmaxf((float)((double)s_inc - mine), 0.f);
      }
      // ---- the decision (Eq. 1 / Eq. 5), the same in every thread
      const double e_tok = (pp.z_tok >= theta) ? pp.e_tok : 0.0;
      const double q_tok = sm.q_tok;
      int accepted;
      if (P.accept_mode == MULO_ACCEPT_THRESHOLD) accepted = e_tok >= P.tau * Z;
      else if (q_tok <= 0.0) accepted = e_tok > 0.0;
      else accepted = uniform24(pp.rnd[0]) * q_tok * Z < e_tok;
      const float invZp = 1.0f / (float)Z;
      if (tid == 0) {
        a.flags[g] = accepted ? 0 : 1;
        if (a.p_tok || a.q_tok || a.accept_prob)
          lane_write_probs(a.p_tok, a.q_tok, a.accept_prob, g, e_tok, q_tok, Z, P.accept_mode == MULO_ACCEPT_THRESHOLD);
      }

      // ---- the draws (one copy of the code: a loop over the draws the position needs).
      // A draw = the thread's sum, a block scan in double, ONE barrier, and the walk of the thread
      // that owns u * total.  Weight of an entry: residual max(0, e / Z_p - q) with q from the draft
      // row's list of this thread (found by popcount on the two masks), or target e; entries below
      // theta weigh nothing.  A residual without mass is drawn again from the target weights with
      // the same uniform.
      const uint32_t t_base = base;
      const int n_lo = __popc(m_lo), nq_lo = __popc(dm_lo);
      int pending = draws_for(P.resample_mode, accepted);   // bit 0 residual, bit 1 target
      bool no_mass = false;
      int dcall = 0;   // consecutive draws alternate between the two scan buffers
#pragma unroll 1
      while (pending) {
        const bool is_res = (pending & kDrawResidual) != 0;
        const bool resid = is_res && !no_mass;
        const double u = uniform24(pp.rnd[is_res ? 1 : 2]);
        int32_t* const out = (is_res ? a.cand_res : a.cand_tgt) + g;
        // The thread's sum needs no pass over its list.  Target weights: the exps of its entries
        // >= theta are known already (s_inc).  Residual: max(0, p - q) = p - min(p, q), and
        // min(p, q) is not zero only for ids that BOTH rows kept, so the sum is s_inc / Z_p minus
        // the min over the intersection of the two masks (about a third of the entries).
        float S = s_inc;
        if (resid) {
          auto both = [&](uint32_t bit, uint32_t m, uint32_t dm, uint32_t tb, uint32_t qb) -> float {
            const uint32_t below = bit - 1u;
            const float z = bit ? lds_f32(tb + (uint32_t)(__popc(m & below) * step)) : -INFINITY;
            const float q = bit ? lds_f32(qb + (uint32_t)(__popc(dm & below) * step)) : 0.f;
            const float pe = __fmul_rn(ex2f(fmaf(z, kLog2e, c0)), invZp);
            return z >= theta ? fminf(pe, q) : 0.f;
          };
          float mins = 0.f;
#pragma unroll 1
          for (int hf = 0; hf < 2; ++hf) {
            const uint32_t m = hf ? m_hi : m_lo, dm = hf ? dm_hi : dm_lo;
            const uint32_t tb = hf ? t_base + (uint32_t)(n_lo * step) : t_base;
            const uint32_t qb = hf ? q_base + (uint32_t)(nq_lo * step) : q_base;
            uint32_t im = m & dm;
            const int trips = (__reduce_max_sync(kFull, __popc(im)) + 1) >> 1;
            for (int it = 0; it < trips; ++it) {   // two entries per trip: their chains overlap
              const uint32_t b0 = im & (0u - im);
              im ^= b0;
              const uint32_t b1 = im & (0u - im);
              im ^= b1;
              const float v0 = both(b0, m, dm, tb, qb), v1 = both(b1, m, dm, tb, qb);
              mins += v0;
              mins += v1;
            }
          }
          S = fmaxf(__fmul_rn(s_inc, invZp) - mins, 0.f);
        }
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
        if (!(total > 0.0)) {   // block-uniform
          if (resid) {
            no_mass = true;   // the same draw again, from the target weights
            continue;
          }
          pending &= ~(is_res ? kDrawResidual : kDrawTarget);
          no_mass = false;
          continue;
        }
        const double y = u * total;
        const double lo = before + excl, hi = before + inc;
        // One thread owns u * total; its WARP walks that thread's entries together: lane k takes the
        // owner's k-th entry (a thread holds at most 32), finds the entry's id by the k-th set bit of
        // the owner's mask, forms its weight, and an inclusive scan in double finds the first entry
        // whose running sum passes y.
        const unsigned own = __ballot_sync(kFull, lo <= y && y < hi);
        if (own) {   // warp-uniform
          const int src = __ffs(own) - 1;
          const uint32_t o_mlo = __shfl_sync(kFull, m_lo, src), o_mhi = __shfl_sync(kFull, m_hi, src);
          const uint32_t o_dlo = __shfl_sync(kFull, dm_lo, src), o_dhi = __shfl_sync(kFull, dm_hi, src);
          const uint32_t o_tb = __shfl_sync(kFull, t_base, src), o_qb = __shfl_sync(kFull, q_base, src);
          const double o_lo = __shfl_sync(kFull, lo, src);
          const int o_nlo = __popc(o_mlo), o_n = o_nlo + __popc(o_mhi);
          const bool have = lane < o_n, upper = lane >= o_nlo;
          const uint32_t mm = upper ? o_mhi : o_mlo, dd = upper ? o_dhi : o_dlo;
          const int pos = have ? (int)__fns(mm, 0u, (upper ? lane - o_nlo : lane) + 1) : 0;
          const uint32_t bit = 1u << pos;
          float w = 0.f;
          if (have) {
            const float z = lds_f32(o_tb + (uint32_t)(lane * step));
            w = ex2f(fmaf(z, kLog2e, c0));
            if (resid) {
              w = __fmul_rn(w, invZp);
              if (dd & bit) {
                const int qi = (upper ? __popc(o_dlo) : 0) + __popc(dd & (bit - 1u));
                w = fmaxf(__fsub_rn(w, lds_f32(o_qb + (uint32_t)(qi * step))), 0.f);
              }
            }
            if (!(z >= theta)) w = 0.f;
          }
          double run = (double)w;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const double v = __shfl_up_sync(kFull, run, o);
            if (lane >= o) run += v;
          }
          const unsigned has = __ballot_sync(kFull, w > 0.f);
          const unsigned hit = __ballot_sync(kFull, w > 0.f && o_lo + run > y);
          // rounding left the sum short: the last entry with weight.  No entry with weight at all:
          // the thread's sum was rounding noise of the difference above (about once in 1e8 draws) --
          // the position goes to the general routines
          const int chosen = hit ? __ffs(hit) - 1 : has ? 31 - __clz(has) : -1;
          if (lane == chosen) *out = ((tid & ~31) + src) * W + (upper ? 32 : 0) + pos;
          if (chosen < 0 && lane == 0) {
            atomicOr(a.dev_status, MULO_DEV_DENSE_FALLBACK);
            defer(g);
          }
        }
        pending &= ~(is_res ? kDrawResidual : kDrawTarget);
        no_mass = false;
      }
    }
  }
#undef rslot
#undef rphase
}

}  // namespace mulo
