// The general ("dense") per-position routine: everything one visit of a target
// grid position computes, working on whole vocabulary rows in global memory.
#pragma once

#include "mulo_device.cuh"
#include "../../include/mulo.h"

namespace mulo {

// per-row statistics of a distribution  prob(x) = [z >= theta] exp(z - m) / Z
struct RowStats {
  float theta, m;
  double Z;
};

// What the kernels need from mulo_params, resolved on the host.
struct DevParams {
  int B, H, W, V, r, h, w;
  int bf16;
  float invT, cfg_scale;
  int top_k;         // 0 = off
  int accept_mode;
  double tau;
  int pool_k;        // <= 1 = off
  double pool_delta;
  int radius, clip, resample_mode;
  uint32_t seed_lo, seed_hi, round, image_offset;
};

// which inverse-CDF draws a visit has to produce
enum : int { kDrawNone = 0, kDrawResidual = 1, kDrawTarget = 2 };

struct PositionOut {   // valid in thread 0 after dense_position
  float p_tok, q_tok, accept_prob;
  int accepted;
  int tok_residual, tok_target;   // -1 when not drawn
};

// Shared memory for pooling: pn[pool_k] doubles then a V-bit map, carved from
// dynamic shared memory by the kernels.
struct PoolSmem {
  double* pn;          // p(n_j), later the inclusive prefix c_j
  uint32_t* bitmap;    // bit x set  <=>  x in A \ {x~}
};

__device__ __forceinline__ float prob_f(float z, float theta, float m, float invZ) {
  return (z >= theta) ? __fmul_rn(expf(__fsub_rn(z, m)), invZ) : 0.0f;
}

// One inverse-CDF draw over w(x) = max(0, p'(x) - lambda q(x)), ascending token
// id: returns min{x : C(x) > u * Z_w} in every thread, or -1 if Z_w == 0.
__device__ inline int dense_draw(const RowSrc& tr, const RowSrc& qr, const RowStats& sp,
                                 const RowStats& sq, float invZp, float invZq, float lambda,
                                 int tok, double w_tok, const uint32_t* bitmap, double u,
                                 BlockScratch& bs) {
  const int V = tr.V;
  const int E = dense_run(V);
  const int beg = (int)threadIdx.x * E;
  const int end = min(V, beg + E);
  float zt[8], zq[8];
  auto weight = [&](int x, float a, float b) -> double {
    if (x == tok) return w_tok;
    float p = prob_f(a, sp.theta, sp.m, invZp);
    if (bitmap && ((bitmap[x >> 5] >> (x & 31)) & 1u)) p = 0.0f;
    float q = prob_f(b, sq.theta, sq.m, invZq);
    float w = __fsub_rn(p, __fmul_rn(lambda, q));
    return (double)fmaxf(w, 0.0f);
  };
  double local = 0.0;
  for (int x = beg; x < end; x += 8) {
    load8(tr, x, zt);
    load8(qr, x, zq);
#pragma unroll
    for (int j = 0; j < 8; ++j) local += weight(x + j, zt[j], zq[j]);
  }
  block_exscan(local, bs);
  const double total = bs.ex[kThreads];
  if (!(total > 0.0)) {
    __syncthreads();
    return -1;
  }
  const double y = u * total;
  if (threadIdx.x == 0) {
    bs.owner = kThreads;
    bs.found = -1;
  }
  __syncthreads();
  if (bs.ex[threadIdx.x + 1] > y) atomicMin(&bs.owner, (int)threadIdx.x);
  __syncthreads();
  if ((int)threadIdx.x == bs.owner) {
    double c = bs.ex[threadIdx.x];
    int pick = -1, last_pos = -1;
    for (int x = beg; x < end && pick < 0; x += 8) {
      load8(tr, x, zt);
      load8(qr, x, zq);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        double wv = weight(x + j, zt[j], zq[j]);
        if (wv > 0.0) last_pos = x + j;
        c += wv;
        if (pick < 0 && c > y) pick = x + j;
      }
    }
    bs.found = pick >= 0 ? pick : last_pos;
  }
  __syncthreads();
  int res = bs.found;
  if (res < 0) {
    // Not reachable in exact arithmetic (u < 1 and the owner's slice has
    // mass); kept so that rounding in the scan can never produce a token
    // without weight: thread 0 walks the whole row.
    if (threadIdx.x == 0) {
      double c = 0.0;
      int pick = -1, last_pos = -1;
      for (int x = 0; x < V && pick < 0; ++x) {
        double wv = weight(x, load1(tr, x), load1(qr, x));
        if (wv > 0.0) last_pos = x;
        c += wv;
        if (c > y) pick = x;
      }
      bs.found = pick >= 0 ? pick : last_pos;
    }
    __syncthreads();
    res = bs.found;
  }
  __syncthreads();
  return res;
}

// Everything for one target position.  `draws` tells which candidates to
// produce when the accept bit is not yet known (kDrawNone: verify only); with
// `decide` false the accept bit is taken from `given_accept` (resample stage).
//   need(draw) is evaluated after the accept decision by `want`.
template <class WantDraws>
__device__ inline void dense_position(const DevParams& P, const RowSrc& tr, const RowSrc& qr,
                                      const RowStats& sq, int tok, const uint16_t* nn,
                                      uint32_t image, uint32_t position, bool decide,
                                      int given_accept, WantDraws want, BlockScratch& bs,
                                      PoolSmem ps, uint32_t* dev_status, PositionOut& out) {
  RowStats sp;
  dense_row_stats(tr, P.top_k, bs, sp.theta, sp.m, sp.Z);
  const float invZp = (float)(1.0 / sp.Z);
  const float invZq = (float)(1.0 / sq.Z);

  // token probabilities in double (thread 0), broadcast
  if (threadIdx.x == 0) {
    float zt = load1(tr, tok), zq = load1(qr, tok);
    double p = (zt >= sp.theta) ? exp((double)zt - (double)sp.m) / sp.Z : 0.0;
    double q = (zq >= sq.theta) ? exp((double)zq - (double)sq.m) / sq.Z : 0.0;
    bs.bd[0] = p;
    bs.bd[1] = q;
    if (q <= 0.0) atomicOr(dev_status, MULO_DEV_ZERO_DRAFT_PROB);
  }
  __syncthreads();
  const double p_tok = bs.bd[0], q_tok = bs.bd[1];
  double mass = p_tok;   // pooled mass P
  const uint32_t* bitmap = nullptr;

  if (P.pool_k > 1) {
    // Eq. 3-4: c_j = sum_{m<=j} p(n_m) along the neighbour list, J = last j of
    // the leading run with c_j < delta; the mass of n_1..n_J moves onto x~.
    const uint16_t* row = nn + (size_t)tok * P.pool_k;
    const int nb = P.pool_k - 1;
    for (int x = threadIdx.x; x < (P.V + 31) / 32; x += kThreads) ps.bitmap[x] = 0u;
    // prefix sums over the list, kThreads entries at a time
    double carry = 0.0;
    int J = 0;
    bool open = true;
    for (int base = 0; base < nb; base += kThreads) {
      const int j = base + (int)threadIdx.x;   // list index j+1
      double pj = 0.0;
      if (j < nb) {
        int id = row[j + 1];
        if (id >= P.V) {
          atomicOr(dev_status, MULO_DEV_BAD_TOKEN);
          id = P.V - 1;
        }
        float zt = load1(tr, id);
        pj = (zt >= sp.theta) ? (double)expf(__fsub_rn(zt, sp.m)) / sp.Z : 0.0;
      }
      block_exscan(pj, bs);
      const double cj = carry + bs.ex[threadIdx.x] + pj;   // inclusive prefix c_{j+1}
      if (j < nb) ps.pn[j] = cj;
      if (threadIdx.x == 0) bs.owner = kThreads;
      __syncthreads();
      if (j < nb && !(cj < P.pool_delta)) atomicMin(&bs.owner, (int)threadIdx.x);
      __syncthreads();
      const int first_bad = bs.owner;   // first index in this tile with c >= delta
      if (open) {
        const int tile = min(kThreads, nb - base);
        if (first_bad >= tile) J = base + tile;
        else {
          J = base + first_bad;
          open = false;
        }
      }
      carry += bs.ex[kThreads];
      __syncthreads();
      if (!open) break;
    }
    __syncthreads();
    if (J > 0) mass = p_tok + ps.pn[J - 1];
    for (int j = threadIdx.x; j < J; j += kThreads) {
      int id = min((int)row[j + 1], P.V - 1);
      atomicOr(&ps.bitmap[id >> 5], 1u << (id & 31));
    }
    __syncthreads();
    bitmap = ps.bitmap;
  }

  // acceptance (Eq. 1 / Eq. 5)
  uint4 rnd = philox4x32_10(make_uint4(position, image, P.round, 0u), make_uint2(P.seed_lo, P.seed_hi));
  double thr;
  int accepted;
  if (P.accept_mode == MULO_ACCEPT_THRESHOLD) {
    thr = mass;
    accepted = mass >= P.tau;
  } else {
    if (q_tok <= 0.0) thr = mass > 0.0 ? 1.0 : 0.0;
    else thr = fmin(1.0, mass / q_tok);
    accepted = uniform24(rnd.x) < thr;
  }
  if (!decide) accepted = given_accept;

  const int draws = want(accepted);
  int t_res = -1, t_tgt = -1;
  if (draws & kDrawResidual) {
    double w_tok = fmax(0.0, mass - q_tok);
    t_res = dense_draw(tr, qr, sp, sq, invZp, invZq, 1.0f, tok, w_tok, bitmap, uniform24(rnd.y), bs);
    if (t_res < 0)   // residual without mass: the lambda = 0 weights, same uniform
      t_res = dense_draw(tr, qr, sp, sq, invZp, invZq, 0.0f, tok, mass, bitmap, uniform24(rnd.y), bs);
  }
  if (draws & kDrawTarget)
    t_tgt = dense_draw(tr, qr, sp, sq, invZp, invZq, 0.0f, tok, mass, bitmap, uniform24(rnd.z), bs);

  out.p_tok = (float)p_tok;
  out.q_tok = (float)q_tok;
  out.accept_prob = (float)thr;
  out.accepted = accepted;
  out.tok_residual = t_res;
  out.tok_target = t_tgt;
}

__device__ __forceinline__ int checked_token(int tok, int V, uint32_t* dev_status) {
  if (tok < 0 || tok >= V) {
    if (threadIdx.x == 0) atomicOr(dev_status, MULO_DEV_BAD_TOKEN);
    tok = min(max(tok, 0), V - 1);
  }
  return tok;
}

// Which draws does a visit need once its accept bit is known (fused round)?
__device__ __forceinline__ int draws_for(int mode, int accepted) {
  int d = 0;
  if (mode == MULO_RESAMPLE_RESIDUAL_ALL || (!accepted && mode != MULO_RESAMPLE_TARGET_ALL)) d |= kDrawResidual;
  if (mode == MULO_RESAMPLE_TARGET_ALL || (accepted && mode != MULO_RESAMPLE_RESIDUAL_ALL) ||
      (!accepted && mode == MULO_RESAMPLE_ISOLATED_RESIDUAL))
    d |= kDrawTarget;
  return d;
}

}  // namespace mulo
