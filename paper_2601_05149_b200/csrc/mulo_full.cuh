// The fast path of the fused round for rows WITHOUT a top-k cut (the paper's default sampling
// setting), when the vocabulary splits evenly over a CTA's 256 threads and the rows of one
// position fit in shared memory.
//
// Without a cut there is nothing to select: every entry of a row is exponentiated once.  A
// persistent CTA owns a contiguous range of parent (low-res) cells.  Per parent it brings the
// draft row into shared memory once (plain bulk copies, never multicast) -- unless the decision
// rule and the resample mode never look at q (Eq. 5 with redraws from the target distribution),
// in which case the draft logits are not read at all -- and then, child by child, the target
// position's conditional and unconditional rows.  Every thread owns a contiguous range of
// W = V / 256 ids of the resident row, so that per-thread sums are slices of the ascending-id CDF:
//
//   softmax      one pass: a running maximum and a sum of exponentials against it per thread
//                (the sum is rescaled on the rare occasions the maximum moves), then the block
//                maximum, the threads' sums rescaled to it, and one block scan in double that
//                gives both the partition sum and the CDF slice of every thread.
//   pooling      Eq. 3-4 on the resident row: the neighbour list of x~ is walked in tiles of 256,
//                prefix masses by a block scan; the pooled ids are marked in a V-bit map and their
//                weights leave their owners' sums through 64-bit fixed-point shared atomics
//                (integer addition: the result does not depend on the order).
//   draws        target weights: the thread sums are known, the owner of u * total walks its W
//                ids.  Residual max(0, p' - q): one more pass over the two resident rows.
//
// The 128-bit shared loads of a warp are spread over the bank groups by starting every thread
// at a different 16-byte piece of its range (sums do not depend on the order; the walk of a
// draw's owner thread is in ascending id).
#pragma once

#include "mulo_lane.cuh"

namespace mulo {

constexpr int kFThreads = 256;
constexpr int kFWarps = kFThreads / 32;
constexpr uint32_t kFPiece = 16384;      // bytes per bulk copy
constexpr float kFix40 = 1099511627776.0f;   // 2^40: fixed-point scale of the pooled weights

struct FullArgs {
  DevParams P;
  const char* cond;
  const char* uncond;
  const char* draft;
  const int32_t* draft_tok_lo;
  const uint16_t* nn;
  float* p_tok;
  float* q_tok;
  float* accept_prob;
  uint8_t* flags;
  int32_t* cand_res;
  int32_t* cand_tgt;
  uint32_t* dev_status;
  int n_parents;
  int W;         // ids per thread
  int need_q;    // 0: neither the decision nor any draw uses the draft distribution
};

struct FullSmem {
  uint64_t bar_q, bar_t;
  double wtot[2][kFWarps];   // block scans; consecutive scans alternate
  double bd[kFWarps];        // block sums
  float bf[2][kFWarps];      // block maxima; consecutive reductions alternate
  uint32_t rnd[3];
  double p_tok, q_tok;       // exp(z - max) of x~ at the current position; q(x~) of the parent
  double cJ;                 // pooled prefix mass c_J
  double pick_w;             // weight of x~ in a draw
  int first_bad;
  int tok;
  int abort;
};

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// z of one 16-byte piece (8 bf16 / 4 fp32 ids) of a resident row
template <bool BF16, bool ROW_U>
__device__ __forceinline__ void full_piece(uint32_t ac, uint32_t au, float s, float invT, float (&z)[BF16 ? 8 : 4]) {
  const uint4 c = lds128(ac);
  uint4 u = make_uint4(0, 0, 0, 0);
  if (ROW_U) u = lds128(au);
  const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, uw[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    if (BF16) {
      z[2 * j] = mix_logit(bf16_lo(cw[j]), bf16_lo(uw[j]), ROW_U, s, invT);
      z[2 * j + 1] = mix_logit(bf16_hi(cw[j]), bf16_hi(uw[j]), ROW_U, s, invT);
    } else {
      z[j] = mix_logit(__uint_as_float(cw[j]), __uint_as_float(uw[j]), ROW_U, s, invT);
    }
  }
}
// The same piece as pairs of ids, with packed fp32 instructions (each half one IEEE rounding, as the
// definition of a pre-processed logit requires: d = c - u; v = fma(s, d, u); z = v * invT)
template <bool BF16, bool ROW_U, bool SCALE>
__device__ __forceinline__ void full_piece2(uint32_t ac, uint32_t au, float2 s2, float2 t2, float2 (&z)[BF16 ? 4 : 2]) {
  const uint4 c = lds128(ac);
  uint4 u = make_uint4(0, 0, 0, 0);
  if (ROW_U) u = lds128(au);
  const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, uw[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int j = 0; j < (BF16 ? 4 : 2); ++j) {
    float2 v, un;
    if (BF16) {
      v = make_float2(bf16_lo(cw[j]), bf16_hi(cw[j]));
      un = make_float2(bf16_lo(uw[j]), bf16_hi(uw[j]));
    } else {
      v = make_float2(__uint_as_float(cw[2 * j]), __uint_as_float(cw[2 * j + 1]));
      un = make_float2(__uint_as_float(uw[2 * j]), __uint_as_float(uw[2 * j + 1]));
    }
    if (ROW_U) v = __ffma2_rn(s2, __ffma2_rn(un, make_float2(-1.f, -1.f), v), un);   // fma(u, -1, c) rounds as c - u
    if (SCALE) v = __fmul2_rn(v, t2);
    z[j] = v;
  }
}
// z of one id of a resident row
template <bool BF16, bool ROW_U>
__device__ __forceinline__ float full_one(const unsigned char* crow, const unsigned char* urow, int x, float s, float invT) {
  float c, u = 0.f;
  if (BF16) {
    c = __uint_as_float((uint32_t) reinterpret_cast<const unsigned short*>(crow)[x] << 16);
    if (ROW_U) u = __uint_as_float((uint32_t) reinterpret_cast<const unsigned short*>(urow)[x] << 16);
  } else {
    c = reinterpret_cast<const float*>(crow)[x];
    if (ROW_U) u = reinterpret_cast<const float*>(urow)[x];
  }
  return mix_logit(c, u, ROW_U, s, invT);
}

template <bool BF16, bool HAS_U>
__global__ void __launch_bounds__(kFThreads, 3) k_round_full(const __grid_constant__ FullArgs a) {
  constexpr int esz = BF16 ? 2 : 4;
  constexpr int N = 16 / esz;   // ids per 16-byte piece
  extern __shared__ __align__(128) unsigned char dyn[];
  __shared__ FullSmem sm;
  const DevParams& P = a.P;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int p_begin = (int)(((long long)a.n_parents * blockIdx.x) / gridDim.x);
  const int p_end = (int)(((long long)a.n_parents * (blockIdx.x + 1)) / gridDim.x);
  if (p_end <= p_begin) return;
  const int V = P.V, W = a.W, nch = W / N, rr = P.r * P.r, NN = P.H * P.W;
  const uint32_t row_bytes = (uint32_t)V * esz;
  const bool need_q = a.need_q != 0, pooling = P.pool_k > 1;
  unsigned char* const qrow = dyn;
  unsigned char* const crow = dyn + (need_q ? row_bytes : 0u);
  unsigned char* const urow = crow + row_bytes;
  uint32_t* const bitmap = reinterpret_cast<uint32_t*>(crow + (HAS_U ? 2u : 1u) * row_bytes);
  unsigned long long* const adj = reinterpret_cast<unsigned long long*>(bitmap + V / 32);
  const uint32_t my_off = (uint32_t)tid * (uint32_t)W * esz;
  const uint32_t q_at = smem_u32(qrow) + my_off, c_at = smem_u32(crow) + my_off, u_at = smem_u32(urow) + my_off;
  const int start = tid % nch;   // this thread's first piece (bank spreading)
  const int id0 = tid * W;

  if (tid == 0) {
    mbar_init(&sm.bar_q, 1);
    mbar_init(&sm.bar_t, 1);
    mbar_fence_init();
    sm.abort = 0;
  }
  __syncthreads();
  uint32_t ph_q = 0, ph_t = 0;

  auto wait = [&](uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return;
    if (*(volatile int*)&sm.abort) return;
#pragma unroll 1
    for (uint32_t it = 0; it < kSpinLimit; ++it)
      if (mbar_try_wait(bar, parity)) return;
    atomicOr(a.dev_status, MULO_DEV_TIMEOUT);
    *(volatile int*)&sm.abort = 1;
  };
  // one thread: a row from global memory into a resident buffer
  auto fetch = [&](unsigned char* dst, const char* src, uint64_t* bar) {
    for (uint32_t o = 0; o < row_bytes; o += kFPiece) {
      const uint32_t n = row_bytes - o < kFPiece ? row_bytes - o : kFPiece;
      bulk_load(dst + o, src + o, n, bar);
    }
  };
  auto fetch_target = [&](size_t g) {   // one thread
    fence_async_smem();
    mbar_expect_tx(&sm.bar_t, HAS_U ? 2u * row_bytes : row_bytes);
    fetch(crow, a.cond + g * (size_t)row_bytes, &sm.bar_t);
    if (HAS_U) fetch(urow, a.uncond + g * (size_t)row_bytes, &sm.bar_t);
  };
  auto position_of = [&](int parent, int child) -> size_t {
    const int hw = P.h * P.w;
    const int b = parent / hw, rem = parent - b * hw, ca = rem / P.w, cc = rem - ca * P.w;
    return (size_t)b * NN + (size_t)(ca * P.r + child / P.r) * P.W + (size_t)(cc * P.r + child % P.r);
  };

  // ---- block helpers (every thread gets the result; fixed order)
  int max_call = 0;
  auto block_max_f = [&](float v) -> float {   // one barrier: consecutive calls alternate buffers
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, o));
    float* const bf = sm.bf[max_call & 1];
    ++max_call;
    if (lane == 0) bf[warp] = v;
    __syncthreads();
    float t = bf[0];
#pragma unroll
    for (int w = 1; w < kFWarps; ++w) t = fmaxf(t, bf[w]);
    return t;
  };
  int scan_call = 0;
  // inclusive scan over the threads in id order: returns the total; `before` = mass of the threads below
  auto block_scan = [&](double v, double& before, double& incl) -> double {
    double inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double n = __shfl_up_sync(kFull, inc, o);
      if (lane >= o) inc += n;
    }
    double* const wt = sm.wtot[scan_call & 1];
    ++scan_call;
    if (lane == 31) wt[warp] = inc;
    __syncthreads();
    double pre = 0.0, total = 0.0;
#pragma unroll
    for (int w = 0; w < kFWarps; ++w) {
      const double x = wt[w];
      if (w == warp) pre = total;
      total += x;
    }
    // (the mass below this thread comes from its neighbour's inclusive sum, not from inc - v,
    // which would cancel the small masses before a large v)
    double exc = __shfl_up_sync(kFull, inc, 1);
    if (lane == 0) exc = 0.0;
    incl = pre + inc;
    before = pre + exc;
    return total;
  };

  // ---- one pass over this thread's part of a resident row: running maximum m and the sum of
  //      2^((z - m) log2 e) against it
  auto softmax_pass_t = [&](auto row_u_tag, auto scale_tag, uint32_t at_c, uint32_t at_u, float s, float& m, float& sum) {
    constexpr bool ROW_U = decltype(row_u_tag)::value;
    constexpr bool SCALE = decltype(scale_tag)::value;
    constexpr int NP = N / 2;   // pairs per piece
    const float2 s2 = make_float2(s, s), t2 = make_float2(P.invT, P.invT), l2 = make_float2(kLog2e, kLog2e);
    m = -INFINITY;
    float2 acc = make_float2(0.f, 0.f);
    int ci = start;
#pragma unroll 1
    for (int i = 0; i < nch; ++i) {
      float2 z[NP];
      full_piece2<BF16, ROW_U, SCALE>(at_c + (uint32_t)ci * 16u, at_u + (uint32_t)ci * 16u, s2, t2, z);
      if (++ci == nch) ci = 0;
      float cm = fmaxf(z[0].x, z[0].y);
#pragma unroll
      for (int j = 1; j < NP; ++j) cm = fmaxf(cm, fmaxf(z[j].x, z[j].y));
      if (cm > m) {
        const float f = ex2f((m - cm) * kLog2e);   // (0 * 2^-inf = 0 on the first piece)
        acc = __fmul2_rn(acc, make_float2(f, f));
        m = cm;
      }
      const float c0 = -m * kLog2e;
      const float2 c2 = make_float2(c0, c0);
#pragma unroll
      for (int j = 0; j < NP; ++j) {
        const float2 t = __ffma2_rn(z[j], l2, c2);
        acc = __fadd2_rn(acc, make_float2(ex2f(t.x), ex2f(t.y)));
      }
    }
    sum = acc.x + acc.y;
  };
  const bool scale = P.invT != 1.0f;
  auto softmax_pass = [&](auto row_u_tag, uint32_t at_c, uint32_t at_u, float s, float& m, float& sum) {
    if (scale) softmax_pass_t(row_u_tag, std::true_type{}, at_c, at_u, s, m, sum);   // block-uniform
    else softmax_pass_t(row_u_tag, std::false_type{}, at_c, at_u, s, m, sum);
  };

  for (int parent = p_begin; parent < p_end; ++parent) {
    // ------------------------------------------------------------ the parent's draft row
    if (tid == 0 && !sm.abort) {
      sm.tok = checked_token(__ldg(a.draft_tok_lo + parent), V, a.dev_status);
      if (need_q) {
        fence_async_smem();
        mbar_expect_tx(&sm.bar_q, row_bytes);
        fetch(qrow, a.draft + (size_t)parent * row_bytes, &sm.bar_q);
      }
      fetch_target(position_of(parent, 0));
    }
    __syncthreads();
    // A wait of this CTA gave up (block-uniform: raised before the last barrier, and nothing was
    // requested since): nothing more is written for its rows; the copy that did not arrive gets a
    // bounded time to land before the shared memory is given up.
    if (*(volatile int*)&sm.abort) {
      for (int i = 0; i < 64; ++i) __nanosleep(1000);
      return;
    }
    const int tok = sm.tok;
    float m_q = 0.f, c0_q = 0.f, invZq = 0.f;
    double q_tok = 0.0;
    if (need_q) {
      wait(&sm.bar_q, ph_q);
      ph_q ^= 1u;
      float mt, st;
      softmax_pass(std::false_type{}, q_at, q_at, 0.f, mt, st);
      m_q = block_max_f(mt);
      c0_q = -m_q * kLog2e;
      const double mine = (double)(st * ex2f((mt - m_q) * kLog2e));
      double before, incl;
      const double Zq = block_scan(mine, before, incl);
      invZq = 1.0f / (float)Zq;
      if (tid == 0) {
        const float zq = full_one<BF16, false>(qrow, qrow, tok, 0.f, P.invT);
        const double q = lane_exp2(((double)zq - (double)m_q) * 1.4426950408889634) / Zq;
        if (q <= 0.0) atomicOr(a.dev_status, MULO_DEV_ZERO_DRAFT_PROB);
        sm.q_tok = q;
      }
      __syncthreads();
      q_tok = sm.q_tok;
    }

    for (int child = 0; child < rr; ++child) {
      const size_t g = position_of(parent, child);
      const int b = (int)(g / (size_t)NN), t = (int)(g - (size_t)b * NN);
      if (tid == 32) {
        const uint4 rnd = lane_philox(make_uint4((uint32_t)t, (uint32_t)b + P.image_offset, P.round, 0u),
                                      make_uint2(P.seed_lo, P.seed_hi));
        sm.rnd[0] = rnd.x;
        sm.rnd[1] = rnd.y;
        sm.rnd[2] = rnd.z;
      }
      wait(&sm.bar_t, ph_t);
      ph_t ^= 1u;
      float mt, st;
      softmax_pass(std::integral_constant<bool, HAS_U>{}, c_at, u_at, P.cfg_scale, mt, st);
      const float M = block_max_f(mt);
      const float c0 = -M * kLog2e;
      const float S_t = st * ex2f((mt - M) * kLog2e);   // this thread's ids, against the row maximum
      const float z_tok = full_one<BF16, HAS_U>(crow, urow, tok, P.cfg_scale, P.invT);
      const float e_tok = ex2f(fmaf(z_tok, kLog2e, c0));
      // exp(z_tok - M) in double by one thread, published by the scan's barrier
      if (tid == 0) sm.p_tok = lane_exp2(((double)z_tok - (double)M) * 1.4426950408889634);
      double before, incl;
      const double Z = block_scan((double)S_t, before, incl);
      const float invZp = 1.0f / (float)Z;

      // ---- Eq. 3-4: the leading run of the neighbour list whose prefix mass stays below delta
      int J = 0;
      double cJ = 0.0;
      if (pooling) {
        // Every thread takes `per` consecutive entries of the neighbour list (at most 8: the list
        // has at most 2047), so one block scan gives every entry's prefix mass.
        const uint16_t* const row = a.nn + (size_t)tok * P.pool_k;
        const int nb = P.pool_k - 1;
        const int per = (nb + kFThreads - 1) / kFThreads;
        const int j0 = tid * per;
        for (int x = tid; x < V / 32; x += kFThreads) bitmap[x] = 0u;
        adj[tid] = 0ull;
        if (tid == 0) sm.first_bad = nb;
        float e[8];
        double mine = 0.0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          e[i] = 0.f;
          if (i < per && j0 + i < nb) {
            int id = __ldg(row + j0 + i + 1);
            if (id >= V) {
              atomicOr(a.dev_status, MULO_DEV_BAD_TOKEN);
              id = V - 1;
            }
            e[i] = ex2f(fmaf(full_one<BF16, HAS_U>(crow, urow, id, P.cfg_scale, P.invT), kLog2e, c0));
            mine += (double)e[i];
          }
        }
        double bef, inc;
        block_scan(mine, bef, inc);   // (its barrier also publishes first_bad and the cleared map)
        // c_j < delta, in units of the partition sum
        const double limit = P.pool_delta * Z;
        {
          double c = bef;
          int bad = nb;
#pragma unroll
          for (int i = 0; i < 8; ++i)
            if (i < per && j0 + i < nb) {
              c += (double)e[i];
              if (bad == nb && !(c < limit)) bad = j0 + i;
            }
          if (bad < nb) atomicMin(&sm.first_bad, bad);
        }
        __syncthreads();
        J = sm.first_bad;   // the leading run n_1 .. n_J keeps its prefix mass below delta
        if (J > 0 && (J - 1) / per == tid) {
          double c = bef;
#pragma unroll
          for (int i = 0; i < 8; ++i)
            if (j0 + i < J) c += (double)e[i];
          sm.cJ = c / Z;
        }
        // the pooled ids: out of the map of drawable ids, their weights out of their owners' sums
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (i < per && j0 + i < J) {
            int id = __ldg(row + j0 + i + 1);
            if (id >= V) id = V - 1;
            const uint32_t bit = 1u << (id & 31);
            const uint32_t old = atomicOr(&bitmap[id >> 5], bit);
            if (!(old & bit) && id != tok)   // (a list may name an id twice, or x~ again)
              atomicAdd(&adj[id / W], __float2ull_rz(e[i] * kFix40));
          }
        __syncthreads();
        if (J > 0) cJ = sm.cJ;
      }
      const double p_tok = sm.p_tok / Z;
      const double mass = p_tok + cJ;   // pooled mass P of Eq. 3

      // ---- the decision (Eq. 1 / Eq. 5), the same in every thread
      double thr;
      int accepted;
      if (P.accept_mode == MULO_ACCEPT_THRESHOLD) {
        thr = mass;
        accepted = mass >= P.tau;
      } else {
        if (q_tok <= 0.0) thr = mass > 0.0 ? 1.0 : 0.0;
        else thr = fmin(1.0, mass / q_tok);
        accepted = uniform24(sm.rnd[0]) < thr;
      }
      if (tid == 0) {
        a.flags[g] = accepted ? 0 : 1;
        if (a.p_tok) a.p_tok[g] = (float)p_tok;
        if (a.q_tok) a.q_tok[g] = (float)q_tok;
        if (a.accept_prob) a.accept_prob[g] = (float)thr;
      }

      // ---- the draws.  Weights of a target draw, in units of 2^((z - M) log2 e): the entry's own,
      // nothing for a pooled id, mass * Z for x~.  Of a residual draw, in units of probability:
      // max(0, p' - q) with the same p'.  A residual without mass is drawn again from the target
      // weights with the same uniform.
      const bool own_tok = tok >= id0 && tok < id0 + W;
      auto weight = [&](int x, bool resid) -> float {   // the owner's walk and the residual pass
        float e = 0.f;
        if (!(pooling && ((bitmap[x >> 5] >> (x & 31)) & 1u)))
          e = ex2f(fmaf(full_one<BF16, HAS_U>(crow, urow, x, P.cfg_scale, P.invT), kLog2e, c0));
        if (!resid) return x == tok ? (float)(mass * Z) : e;
        if (x == tok) return (float)fmax(0.0, mass - q_tok);
        const float q = __fmul_rn(ex2f(fmaf(full_one<BF16, false>(qrow, qrow, x, 0.f, P.invT), kLog2e, c0_q)), invZq);
        return fmaxf(__fsub_rn(__fmul_rn(e, invZp), q), 0.f);
      };
      int pending = draws_for(P.resample_mode, accepted);
      bool no_mass = false;
#pragma unroll 1
      while (pending) {
        const bool is_res = (pending & kDrawResidual) != 0;
        const bool resid = is_res && !no_mass;
        const double u = uniform24(sm.rnd[is_res ? 1 : 2]);
        int32_t* const out = (is_res ? a.cand_res : a.cand_tgt) + g;
        double S;
        if (!resid) {
          S = (double)S_t;
          if (pooling) S -= (double)adj[tid] * (1.0 / (double)kFix40);
          if (own_tok) S += mass * Z - (double)e_tok;
          S = fmax(S, 0.0);
        } else {
          float acc = 0.f;
          int ci = start;
#pragma unroll 1
          for (int i = 0; i < nch; ++i) {
            const int x0 = id0 + ci * N;
            if (++ci == nch) ci = 0;
#pragma unroll
            for (int j = 0; j < N; ++j) acc += weight(x0 + j, true);
          }
          S = (double)acc;
        }
        double bef, inc;
        const double total = block_scan(S, bef, inc);
        if (!(total > 0.0)) {   // block-uniform
          if (resid) {
            no_mass = true;
            continue;
          }
          pending &= ~(is_res ? kDrawResidual : kDrawTarget);
          no_mass = false;
          continue;
        }
        const double y = u * total;
        // One thread owns u * total; its WARP walks that thread's ids together, 32 at a time in
        // ascending order: weights, an inclusive scan in double, the first id whose running sum
        // passes y.
        const unsigned owner_mask = __ballot_sync(kFull, bef <= y && y < inc);
        if (owner_mask) {   // warp-uniform
          const int src = __ffs(owner_mask) - 1;
          const int o_id0 = __shfl_sync(kFull, id0, src);
          double c = __shfl_sync(kFull, bef, src);
          int pick = -1, last_pos = -1;
          for (int x0 = o_id0; x0 < o_id0 + W && pick < 0; x0 += 32) {
            const int x = x0 + lane;
            const float w = x < o_id0 + W ? weight(x, resid) : 0.f;
            double run = (double)w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
              const double n = __shfl_up_sync(kFull, run, o);
              if (lane >= o) run += n;
            }
            const unsigned has = __ballot_sync(kFull, w > 0.f);
            const unsigned hit = __ballot_sync(kFull, w > 0.f && c + run > y);
            if (has) last_pos = x0 + 31 - __clz(has);
            if (hit) pick = x0 + __ffs(hit) - 1;
            c += __shfl_sync(kFull, run, 31);
          }
          // (rounding left the walk short of y: the last id with weight; none at all cannot be,
          // the thread's sum being positive -- then the thread's first id stands in)
          if (lane == 0) *out = pick >= 0 ? pick : last_pos >= 0 ? last_pos : o_id0;
        }
        pending &= ~(is_res ? kDrawResidual : kDrawTarget);
        no_mass = false;
      }

      __syncthreads();   // everybody is done with the resident target row
      if (tid == 0 && child + 1 < rr && !sm.abort) fetch_target(position_of(parent, child + 1));
    }
  }
}

}  // namespace mulo
