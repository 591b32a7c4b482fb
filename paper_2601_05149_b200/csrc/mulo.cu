// libmulo: kernels and C ABI of the MuLo-SD draft-and-verify round (sm_100a).
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <mutex>
#include <new>
#include <vector>

#include "../../include/mulo.h"
#include "mulo_dense.cuh"
#include "mulo_islands.cuh"
#include "mulo_lane.cuh"
#include "mulo_full.cuh"
#include "mulo_stream.cuh"

using namespace mulo;

// ============================================================== row kernels

struct RowKernelArgs {
  DevParams P;
  const char* cond;
  const char* uncond;
  const char* draft;
  const int32_t* draft_tok_lo;   // fused / upsample: [B,h,w]
  const int32_t* draft_tok_hi;   // unfused verify / resample: [B,H,W]
  const float* stats_in;         // unfused: [B,h,w,4]
  const uint16_t* nn;
  const uint32_t* reject_bits;   // resample stage
  const uint32_t* expand_bits;   // resample stage
  // outputs
  float* p_tok;
  float* q_tok;
  float* accept_prob;
  uint8_t* flags;                // workspace: 1 = rejected
  int32_t* cand_res;             // workspace
  int32_t* cand_tgt;             // workspace
  int32_t* out_tok;              // resample stage
  int32_t* tok_hi_out;           // upsample stage
  float* stats_out;              // upsample stage
  float* q_tok_hi_out;           // upsample stage
  uint32_t* dev_status;
};

__device__ __forceinline__ RowSrc target_row(const RowKernelArgs& a, size_t row) {
  const size_t bytes = (size_t)a.P.V * (a.P.bf16 ? 2 : 4);
  RowSrc r;
  r.cond = a.cond + row * bytes;
  r.uncond = a.uncond ? a.uncond + row * bytes : nullptr;
  r.s = a.P.cfg_scale;
  r.invT = a.P.invT;
  r.V = a.P.V;
  r.bf16 = a.P.bf16;
  return r;
}
__device__ __forceinline__ RowSrc draft_row(const RowKernelArgs& a, size_t cell) {
  const size_t bytes = (size_t)a.P.V * (a.P.bf16 ? 2 : 4);
  RowSrc r;
  r.cond = a.draft + cell * bytes;
  r.uncond = nullptr;
  r.s = 0.f;
  r.invT = a.P.invT;
  r.V = a.P.V;
  r.bf16 = a.P.bf16;
  return r;
}

__device__ __forceinline__ PoolSmem carve_pool(const DevParams& P, unsigned char* dyn) {
  PoolSmem ps;
  ps.pn = reinterpret_cast<double*>(dyn);
  ps.bitmap = reinterpret_cast<uint32_t*>(dyn + (size_t)max(P.pool_k, 1) * sizeof(double));
  return ps;
}

// mulo_upsample_pool: one CTA per low-res cell.
__global__ void __launch_bounds__(kThreads) k_upsample_pool(RowKernelArgs a) {
  __shared__ BlockScratch bs;
  const DevParams& P = a.P;
  const int cell = blockIdx.x;   // b*h*w + ca*w + cc
  const int b = cell / (P.h * P.w), rem = cell % (P.h * P.w), ca = rem / P.w, cc = rem % P.w;
  RowSrc qr = draft_row(a, cell);
  RowStats sq;
  dense_row_stats(qr, P.top_k, bs, sq.theta, sq.m, sq.Z);
  if (threadIdx.x == 0) {
    const int tok = checked_token(a.draft_tok_lo[cell], P.V, a.dev_status);
    const float Zhi = (float)sq.Z, Zlo = (float)(sq.Z - (double)Zhi);
    a.stats_out[(size_t)cell * 4 + 0] = sq.theta;
    a.stats_out[(size_t)cell * 4 + 1] = sq.m;
    a.stats_out[(size_t)cell * 4 + 2] = Zhi;
    a.stats_out[(size_t)cell * 4 + 3] = Zlo;
    float zq = load1(qr, tok);
    double q = (zq >= sq.theta) ? exp((double)zq - (double)sq.m) / ((double)Zhi + (double)Zlo) : 0.0;
    for (int di = 0; di < P.r; ++di)
      for (int dj = 0; dj < P.r; ++dj) {
        size_t t = ((size_t)b * P.H + (size_t)ca * P.r + di) * P.W + (size_t)cc * P.r + dj;
        a.tok_hi_out[t] = a.draft_tok_lo[cell];
        a.q_tok_hi_out[t] = (float)q;
      }
  }
}

// The drafter's own draw (Sec. 3.2 Step 1) for one low-res cell by the general routines:
// q = softmax(topk(l_q / T)), inverse CDF with word 0 of the tag-1 Philox stream.
__device__ inline void sample_cell(const RowKernelArgs& a, int cell, BlockScratch& bs) {
  const DevParams& P = a.P;
  const int b = cell / (P.h * P.w), rem = cell % (P.h * P.w);
  RowSrc qr = draft_row(a, cell);
  RowStats sq;
  dense_row_stats(qr, P.top_k, bs, sq.theta, sq.m, sq.Z);
  __syncthreads();
  const float invZ = (float)(1.0 / sq.Z);
  const uint4 rnd = philox4x32_10(make_uint4((uint32_t)rem, (uint32_t)b + P.image_offset, P.round, 1u),
                                  make_uint2(P.seed_lo, P.seed_hi));
  // lambda = 0 and no special token: the weights are q itself
  const int tok = dense_draw(qr, qr, sq, sq, invZ, invZ, 0.0f, -1, 0.0, nullptr, uniform24(rnd.x), bs);
  if (threadIdx.x == 0) a.out_tok[cell] = tok;
}

// mulo_sample_draft, general path: one CTA per low-res cell.
__global__ void __launch_bounds__(kThreads) k_sample_draft(RowKernelArgs a) {
  __shared__ BlockScratch bs;
  sample_cell(a, blockIdx.x, bs);
}

// Second launch of mulo_sample_draft's fast path: the cells the streaming kernel put on its list.
__global__ void __launch_bounds__(kThreads) k_sample_failed(RowKernelArgs a, const int32_t* fail_list,
                                                            const uint32_t* fail_count) {
  __shared__ BlockScratch bs;
  const size_t total = (size_t)a.P.B * a.P.h * a.P.w;
  const size_t n = min((size_t)*fail_count, total);
  for (size_t idx = blockIdx.x; idx < n; idx += gridDim.x) {
    const size_t cell = (size_t)fail_list[idx];
    if (cell < total) sample_cell(a, (int)cell, bs);
    __syncthreads();
  }
}

// ---- the redraw of R_X, one launch per sequential step (Sec. 3.4, Algorithm 1 Step 6)
// Plan: the positions sorted by their step -- count, scan, fill.  offsets[s] is where step s starts in
// pos_list (s = 1 .. max_step, offsets[max_step + 1] the end); the cursors live behind the offsets.
constexpr int kScanThreads = 1024;

__global__ void __launch_bounds__(256) k_redraw_count(const int32_t* __restrict__ step, int n, int max_step,
                                                      int32_t* cursor) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const int s = step[i];
    if (s >= 1 && s <= max_step) atomicAdd(&cursor[s], 1);
  }
}

__global__ void __launch_bounds__(kScanThreads) k_redraw_scan(int max_step, int32_t* offsets, int32_t* cursor) {
  __shared__ int warp_tot[kScanThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = max_step + 1;                       // entries 0 .. max_step (entry 0 counts nothing)
  const int per = (n + kScanThreads - 1) / kScanThreads;
  const int beg = min(n, tid * per), end = min(n, beg + per);
  int mine = 0;
  for (int i = beg; i < end; ++i) mine += i == 0 ? 0 : cursor[i];
  int inc = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(kFull, inc, o);
    if (lane >= o) inc += v;
  }
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  int pre = 0;
  for (int w = 0; w < warp; ++w) pre += warp_tot[w];
  int run = pre + inc - mine;                        // positions with a step below this thread's first
  for (int i = beg; i < end; ++i) {
    const int c = i == 0 ? 0 : cursor[i];
    offsets[i] = run;
    cursor[i] = run;
    run += c;
  }
  if (tid == kScanThreads - 1) offsets[max_step + 1] = pre + inc;   // (the last thread's inclusive sum: the total)
}

__global__ void __launch_bounds__(256) k_redraw_fill(const int32_t* __restrict__ step, int n, int max_step,
                                                     int32_t* cursor, int32_t* pos_list) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const int s = step[i];
    if (s >= 1 && s <= max_step) pos_list[atomicAdd(&cursor[s], 1)] = i;
  }
}

struct RedrawArgs {
  DevParams P;
  const char* cond;
  const char* uncond;
  const int32_t* pos_list;
  const int32_t* offsets;
  int32_t* out_tok;
  int s;
};

// One step: every position of the step's slice of the list draws its token from the target
// distribution of the given logits; uniform = word 0 of Philox at (t, image, round, 1 + s).
__global__ void __launch_bounds__(kThreads) k_redraw_step(RedrawArgs a) {
  __shared__ BlockScratch bs;
  const DevParams& P = a.P;
  const int beg = a.offsets[a.s], end = a.offsets[a.s + 1];
  const size_t N = (size_t)P.H * P.W, total = (size_t)P.B * N;
  const size_t bytes = (size_t)P.V * (P.bf16 ? 2 : 4);
  for (int i = beg + (int)blockIdx.x; i < end; i += (int)gridDim.x) {
    const size_t g = (size_t)a.pos_list[i];
    if (g < total) {   // block-uniform
      const uint32_t b = (uint32_t)(g / N), t = (uint32_t)(g - (size_t)b * N);
      RowSrc tr;
      tr.cond = a.cond + g * bytes;
      tr.uncond = a.uncond ? a.uncond + g * bytes : nullptr;
      tr.s = P.cfg_scale;
      tr.invT = P.invT;
      tr.V = P.V;
      tr.bf16 = P.bf16;
      RowStats sp;
      dense_row_stats(tr, P.top_k, bs, sp.theta, sp.m, sp.Z);
      __syncthreads();
      const float invZ = (float)(1.0 / sp.Z);
      const uint4 rnd = philox4x32_10(make_uint4(t, b + P.image_offset, P.round, 1u + (uint32_t)a.s),
                                      make_uint2(P.seed_lo, P.seed_hi));
      const int tok = dense_draw(tr, tr, sp, sp, invZ, invZ, 0.0f, -1, 0.0, nullptr, uniform24(rnd.x), bs);
      if (threadIdx.x == 0) a.out_tok[g] = tok;
    }
    __syncthreads();
  }
}

// mulo_downsample: one thread per low-res cell; the most frequent token of its r x r block,
// ties to the one that comes first in raster order of the block (Step 7 stand-in).
__global__ void __launch_bounds__(256) k_downsample(const int32_t* __restrict__ x, int32_t* __restrict__ y,
                                                    int cells, int h, int w, int W, int r) {
  const int cell = blockIdx.x * blockDim.x + threadIdx.x;
  if (cell >= cells) return;
  const int b = cell / (h * w), rem = cell % (h * w), ca = rem / w, cc = rem % w;
  const int32_t* blk = x + ((size_t)b * h * r + (size_t)ca * r) * W + (size_t)cc * r;
  int best_tok = -1, best_count = 0;
  for (int s1 = 0; s1 < r * r; ++s1) {
    const int tok = blk[(size_t)(s1 / r) * W + s1 % r];
    int count = 0;
    for (int s2 = 0; s2 < r * r; ++s2) count += blk[(size_t)(s2 / r) * W + s2 % r] == tok;
    if (count > best_count) {
      best_count = count;
      best_tok = tok;
    }
  }
  y[cell] = best_tok;
}

// mulo_verify (FUSED = false): one CTA per target position, draft statistics given.
// mulo_round  (FUSED = true):  one CTA per low-res cell: draft statistics, then its
// r*r children; accept flags and candidate draws go to the workspace.
template <bool FUSED>
__global__ void __launch_bounds__(kThreads) k_verify_rows(RowKernelArgs a) {
  __shared__ BlockScratch bs;
  extern __shared__ __align__(16) unsigned char dyn[];
  const DevParams& P = a.P;
  PoolSmem ps = carve_pool(P, dyn);
  const int N = P.H * P.W;
  if (FUSED) {
    const int cell = blockIdx.x;
    const int b = cell / (P.h * P.w), rem = cell % (P.h * P.w), ca = rem / P.w, cc = rem % P.w;
    RowSrc qr = draft_row(a, cell);
    RowStats sq;
    dense_row_stats(qr, P.top_k, bs, sq.theta, sq.m, sq.Z);
    {   // the unfused path stores Z_q as an fp32 (hi, lo) pair; keep both paths identical
      const float Zhi = (float)sq.Z, Zlo = (float)(sq.Z - (double)Zhi);
      sq.Z = (double)Zhi + (double)Zlo;
    }
    const int tok = checked_token(a.draft_tok_lo[cell], P.V, a.dev_status);
    for (int di = 0; di < P.r; ++di)
      for (int dj = 0; dj < P.r; ++dj) {
        const int t = (ca * P.r + di) * P.W + cc * P.r + dj;
        const size_t g = (size_t)b * N + t;
        RowSrc tr = target_row(a, g);
        PositionOut o;
        const int mode = P.resample_mode;
        dense_position(P, tr, qr, sq, tok, a.nn, (uint32_t)b + P.image_offset, (uint32_t)t, true, 0,
                       [mode](int acc) { return draws_for(mode, acc); }, bs, ps, a.dev_status, o);
        if (threadIdx.x == 0) {
          a.flags[g] = o.accepted ? 0 : 1;
          a.cand_res[g] = o.tok_residual;
          a.cand_tgt[g] = o.tok_target;
          if (a.p_tok) a.p_tok[g] = o.p_tok;
          if (a.q_tok) a.q_tok[g] = o.q_tok;
          if (a.accept_prob) a.accept_prob[g] = o.accept_prob;
        }
        __syncthreads();
      }
  } else {
    const size_t g = blockIdx.x;
    const int b = (int)(g / N), t = (int)(g % N), i = t / P.W, j = t % P.W;
    const size_t cell = ((size_t)b * P.h + i / P.r) * P.w + j / P.r;
    RowSrc qr = draft_row(a, cell);
    RowStats sq;
    sq.theta = a.stats_in[cell * 4 + 0];
    sq.m = a.stats_in[cell * 4 + 1];
    sq.Z = (double)a.stats_in[cell * 4 + 2] + (double)a.stats_in[cell * 4 + 3];
    const int tok = checked_token(a.draft_tok_hi[g], P.V, a.dev_status);
    RowSrc tr = target_row(a, g);
    PositionOut o;
    dense_position(P, tr, qr, sq, tok, a.nn, (uint32_t)b + P.image_offset, (uint32_t)t, true, 0,
                   [](int) { return (int)kDrawNone; }, bs, ps, a.dev_status, o);
    if (threadIdx.x == 0) {
      a.flags[g] = o.accepted ? 0 : 1;
      a.p_tok[g] = o.p_tok;
      a.q_tok[g] = o.q_tok;
      a.accept_prob[g] = o.accept_prob;
    }
  }
}

// Second launch of mulo_round's fast path: the positions the streaming kernel put on its
// list (rows whose pivot prediction failed), done by the dense routines, one CTA at a time.
__global__ void __launch_bounds__(kThreads) k_verify_failed(RowKernelArgs a, const int32_t* fail_list,
                                                            const uint32_t* fail_count) {
  __shared__ BlockScratch bs;
  extern __shared__ __align__(16) unsigned char dyn[];
  const DevParams& P = a.P;
  PoolSmem ps = carve_pool(P, dyn);
  const int N = P.H * P.W;
  const size_t total = (size_t)P.B * N;
  const size_t n = min((size_t)*fail_count, total);
  for (size_t idx = blockIdx.x; idx < n; idx += gridDim.x) {
    const size_t g = (size_t)fail_list[idx];
    if (g >= total) continue;
    const int b = (int)(g / N), t = (int)(g % N), i = t / P.W, j = t % P.W;
    const size_t cell = ((size_t)b * P.h + i / P.r) * P.w + j / P.r;
    RowSrc qr = draft_row(a, cell);
    RowStats sq;
    dense_row_stats(qr, P.top_k, bs, sq.theta, sq.m, sq.Z);
    {   // Z_q rounded as everywhere else (fp32 hi + lo)
      const float Zhi = (float)sq.Z, Zlo = (float)(sq.Z - (double)Zhi);
      sq.Z = (double)Zhi + (double)Zlo;
    }
    const int tok = checked_token(a.draft_tok_lo[cell], P.V, a.dev_status);
    RowSrc tr = target_row(a, g);
    PositionOut o;
    const int mode = P.resample_mode;
    dense_position(P, tr, qr, sq, tok, a.nn, (uint32_t)b + P.image_offset, (uint32_t)t, true, 0,
                   [mode](int acc) { return draws_for(mode, acc); }, bs, ps, a.dev_status, o);
    if (threadIdx.x == 0) {
      a.flags[g] = o.accepted ? 0 : 1;
      a.cand_res[g] = o.tok_residual;
      a.cand_tgt[g] = o.tok_target;
      if (a.p_tok) a.p_tok[g] = o.p_tok;
      if (a.q_tok) a.q_tok[g] = o.q_tok;
      if (a.accept_prob) a.accept_prob[g] = o.accept_prob;
    }
    __syncthreads();
  }
}

__device__ __forceinline__ int get_bit(const uint32_t* bits, int Ww, int H, int b, int i, int j) {
  return (bits[((size_t)b * H + i) * Ww + (j >> 5)] >> (j & 31)) & 1u;
}

// Would position (i,j), if it had been accepted, have been swept into R_X by
// another rejection?  (some other rejected position within radius l, and -- with
// clipping -- (i,j) is not the image's first rejection)
__device__ __forceinline__ bool covered_by_other(const uint32_t* rej, int Ww, int H, int W, int b, int i,
                                                 int j, int l, int clip, int t0) {
  if (clip && i * W + j == t0) return false;
  for (int ii = max(0, i - l); ii <= min(H - 1, i + l); ++ii)
    for (int jj = max(0, j - l); jj <= min(W - 1, j + l); ++jj)
      if ((ii != i || jj != j) && get_bit(rej, Ww, H, b, ii, jj)) return true;
  return false;
}

// mulo_resample: one CTA per target position; positions outside R_X copy x~.
__global__ void __launch_bounds__(kThreads) k_resample_rows(RowKernelArgs a) {
  __shared__ BlockScratch bs;
  extern __shared__ __align__(16) unsigned char dyn[];
  const DevParams& P = a.P;
  PoolSmem ps = carve_pool(P, dyn);
  const int N = P.H * P.W, Ww = (P.W + 31) / 32;
  const size_t g = blockIdx.x;
  const int b = (int)(g / N), t = (int)(g % N), i = t / P.W, j = t % P.W;
  const int tok_raw = a.draft_tok_hi[g];
  if (!get_bit(a.expand_bits, Ww, P.H, b, i, j)) {
    if (threadIdx.x == 0) a.out_tok[g] = tok_raw;
    return;
  }
  const int rejected = get_bit(a.reject_bits, Ww, P.H, b, i, j);
  int use_res;
  if (P.resample_mode == MULO_RESAMPLE_RESIDUAL_ALL) use_res = 1;
  else if (P.resample_mode == MULO_RESAMPLE_TARGET_ALL) use_res = 0;
  else if (P.resample_mode == MULO_RESAMPLE_ISOLATED_RESIDUAL) {
    use_res = rejected;
    if (rejected) {
      // first rejection of the image: scan the words of image b (uniform across the CTA)
      int t0 = N;
      for (int w = 0; w < P.H * Ww && t0 == N; ++w) {
        uint32_t v = a.reject_bits[(size_t)b * P.H * Ww + w];
        if (v) t0 = (w / Ww) * P.W + (w % Ww) * 32 + __ffs(v) - 1;
      }
      if (covered_by_other(a.reject_bits, Ww, P.H, P.W, b, i, j, P.radius, P.clip, t0)) use_res = 0;
    }
  } else use_res = rejected;
  const size_t cell = ((size_t)b * P.h + i / P.r) * P.w + j / P.r;
  RowSrc qr = draft_row(a, cell);
  RowStats sq;
  sq.theta = a.stats_in[cell * 4 + 0];
  sq.m = a.stats_in[cell * 4 + 1];
  sq.Z = (double)a.stats_in[cell * 4 + 2] + (double)a.stats_in[cell * 4 + 3];
  const int tok = checked_token(tok_raw, P.V, a.dev_status);
  RowSrc tr = target_row(a, g);
  PositionOut o;
  const int draw = use_res ? kDrawResidual : kDrawTarget;
  dense_position(P, tr, qr, sq, tok, a.nn, (uint32_t)b + P.image_offset, (uint32_t)t, false, !rejected,
                 [draw](int) { return draw; }, bs, ps, a.dev_status, o);
  if (threadIdx.x == 0) a.out_tok[g] = use_res ? o.tok_residual : o.tok_target;
}

// ============================================================= mask kernel
// One CTA per image, warps over 32-position tiles: ballot packs accept flags
// into row words, ffs/popc give t_0 and the counts, funnel shifts dilate.

struct MaskArgs {
  int H, W, r, radius, clip, resample_mode;
  const uint8_t* flags;          // [B,H,W] 1 = rejected           (MODE 0, 2)
  const uint32_t* reject_in;     // [B,H,Ww]                        (MODE 1)
  const int32_t* first_in;       // [B]                             (MODE 1)
  uint32_t* reject_bits;         // out (MODE 0, 2)
  uint32_t* expand_bits;         // out (MODE 1, 2)
  int32_t* n_reject;             // out (MODE 0, 2), may be null
  int32_t* first_reject;         // out (MODE 0, 2), may be null
  int32_t* n_expand;             // out (MODE 1, 2), may be null
  const int32_t* cand_res;       // MODE 2
  const int32_t* cand_tgt;       // MODE 2
  const int32_t* draft_tok_lo;   // MODE 2: [B,h,w]
  int32_t* out_tok;              // MODE 2
};

constexpr int kMaskThreads = 256;

// MODE 0: flags -> reject bits, counts, t_0            (tail of mulo_verify)
// MODE 1: reject bits -> expand bits, count            (mulo_local_reject_expand)
// MODE 2: flags -> both masks, counts, output tokens   (tail of mulo_round)
template <int MODE>
__global__ void __launch_bounds__(kMaskThreads) k_mask(MaskArgs a) {
  extern __shared__ uint32_t words[];
  const int H = a.H, W = a.W, Ww = (W + 31) / 32, nw = H * Ww, N = H * W;
  uint32_t* rej = words;
  uint32_t* hd = words + nw;
  uint32_t* ex = words + 2 * nw;
  __shared__ int s_nrej, s_first, s_nexp;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    s_nrej = 0;
    s_first = N;
    s_nexp = 0;
  }
  __syncthreads();
  if (MODE == 1) {
    for (int w = tid; w < nw; w += kMaskThreads) rej[w] = a.reject_in[(size_t)b * nw + w];
    if (tid == 0) s_first = a.first_in[b];
  } else {
    for (int w = warp; w < nw; w += kMaskThreads / 32) {
      const int i = w / Ww, j = (w % Ww) * 32 + lane;
      const bool r = j < W && a.flags[(size_t)b * N + (size_t)i * W + j] != 0;
      const uint32_t word = __ballot_sync(kFull, r);
      if (lane == 0) {
        rej[w] = word;
        if (word) {
          atomicAdd(&s_nrej, __popc(word));
          atomicMin(&s_first, i * W + (w % Ww) * 32 + __ffs(word) - 1);
        }
      }
    }
  }
  __syncthreads();
  const int t0 = s_first;
  if (MODE != 1) {
    for (int w = tid; w < nw; w += kMaskThreads) a.reject_bits[(size_t)b * nw + w] = rej[w];
    if (tid == 0) {
      if (a.n_reject) a.n_reject[b] = s_nrej;
      if (a.first_reject) a.first_reject[b] = t0;
    }
  }
  if (MODE == 0) return;

  // horizontal dilation by l: OR of the row shifted by -l..l, with carries
  // across word boundaries (l <= 31, so only the two adjacent words matter)
  const int l = a.radius;
  for (int w = tid; w < nw; w += kMaskThreads) {
    const int wj = w % Ww;
    const uint32_t cur = rej[w];
    const uint32_t prev = wj > 0 ? rej[w - 1] : 0u;
    const uint32_t next = wj + 1 < Ww ? rej[w + 1] : 0u;
    uint32_t acc = cur;
    for (int s = 1; s <= l; ++s) {
      acc |= __funnelshift_l(prev, cur, s);   // bits moved towards higher j
      acc |= __funnelshift_r(cur, next, s);   // bits moved towards lower j
    }
    if (wj == Ww - 1 && (W & 31)) acc &= (1u << (W & 31)) - 1u;
    hd[w] = acc;
  }
  __syncthreads();
  // vertical dilation, then Eq. 6's clause u >= t_0
  for (int w = tid; w < nw; w += kMaskThreads) {
    const int i = w / Ww, wj = w % Ww;
    uint32_t acc = 0u;
    for (int ii = max(0, i - l); ii <= min(H - 1, i + l); ++ii) acc |= hd[ii * Ww + wj];
    if (a.clip) {
      const int i0 = t0 / W, j0 = t0 % W;
      if (t0 >= N || i < i0) acc = (t0 >= N) ? acc : 0u;
      else if (i == i0) {
        const int lo = j0 - wj * 32;   // first kept bit of this word
        if (lo >= 32) acc = 0u;
        else if (lo > 0) acc &= ~((1u << lo) - 1u);
      }
    }
    ex[w] = acc;
    a.expand_bits[(size_t)b * nw + w] = acc;
    if (acc) atomicAdd(&s_nexp, __popc(acc));
  }
  __syncthreads();
  if (tid == 0 && a.n_expand) a.n_expand[b] = s_nexp;
  if (MODE != 2) return;

  // output assembly: x~ outside R_X, the position's draw inside
  const int h = H / a.r, w_lo = W / a.r;
  for (int t = tid; t < N; t += kMaskThreads) {
    const int i = t / W, j = t % W;
    const size_t g = (size_t)b * N + t;
    int tok = a.draft_tok_lo[((size_t)b * h + i / a.r) * w_lo + j / a.r];
    if ((ex[i * Ww + (j >> 5)] >> (j & 31)) & 1u) {
      const int rejected = (rej[i * Ww + (j >> 5)] >> (j & 31)) & 1u;
      int use_res;
      if (a.resample_mode == MULO_RESAMPLE_RESIDUAL_ALL) use_res = 1;
      else if (a.resample_mode == MULO_RESAMPLE_TARGET_ALL) use_res = 0;
      else if (a.resample_mode == MULO_RESAMPLE_ISOLATED_RESIDUAL)
        use_res = rejected && !covered_by_other(rej, Ww, H, W, 0, i, j, l, a.clip, t0);
      else use_res = rejected;
      tok = use_res ? a.cand_res[g] : a.cand_tgt[g];
    }
    a.out_tok[g] = tok;
  }
}

// ================================================================ host side

struct mulo_ctx {
  int device;
  int sm_count;
  int smem_optin;
  void* ws;
  size_t ws_bytes;
  uint64_t launches;
  std::vector<cudaEvent_t> ev;   // start/stop pairs around the fused row kernel
  size_t ev_used;
  int force_dense;               // diagnostics: never take the fast top-k path
  int no_lane;                   // diagnostics: never take the lane-private kernel
};

static const size_t kStatusBytes = 256;

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static mulo_status validate(const mulo_params* p) {
  if (!p) return MULO_ERR_INVALID_ARG;
  if (p->B < 0 || p->H <= 0 || p->W <= 0 || p->r <= 0) return MULO_ERR_INVALID_ARG;
  if (p->H % p->r || p->W % p->r) return MULO_ERR_INVALID_ARG;
  if (p->V <= 0 || p->V % 8) return MULO_ERR_INVALID_ARG;
  if (p->logit_dtype != MULO_F32 && p->logit_dtype != MULO_BF16) return MULO_ERR_INVALID_ARG;
  if (!(p->temperature > 0.0f) || !isfinite(p->temperature)) return MULO_ERR_INVALID_ARG;
  if (!isfinite(p->cfg_scale)) return MULO_ERR_INVALID_ARG;
  if (p->accept_mode != MULO_ACCEPT_RATIO && p->accept_mode != MULO_ACCEPT_THRESHOLD) return MULO_ERR_INVALID_ARG;
  if (p->resample_mode < 0 || p->resample_mode > MULO_RESAMPLE_ISOLATED_RESIDUAL) return MULO_ERR_INVALID_ARG;
  if (p->radius < 0) return MULO_ERR_INVALID_ARG;
  if (p->pool_k > 1 && !(p->pool_delta >= 0.0f)) return MULO_ERR_INVALID_ARG;
  if (p->V > 65536) return MULO_ERR_UNSUPPORTED;
  if (p->radius > 31) return MULO_ERR_UNSUPPORTED;
  if (p->pool_k > 2048 || p->pool_k > p->V) return MULO_ERR_UNSUPPORTED;
  if ((size_t)p->H * ((p->W + 31) / 32) > 4000) return MULO_ERR_UNSUPPORTED;
  if ((double)p->B * p->H * p->W > 2.0e9) return MULO_ERR_UNSUPPORTED;
  return MULO_OK;
}

static bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

// Kernels are launched on the calling thread's current device, while limits, workspace and the
// built-in scratch array belong to the context's device: the two must be the same.
static mulo_status on_context_device(const mulo_ctx* ctx) {
  if (!ctx) return MULO_ERR_INVALID_ARG;
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess) {
    cudaGetLastError();
    return MULO_ERR_CUDA;
  }
  return cur == ctx->device ? MULO_OK : MULO_ERR_INVALID_ARG;
}

static DevParams to_dev(const mulo_params* p) {
  DevParams d;
  d.B = p->B; d.H = p->H; d.W = p->W; d.V = p->V; d.r = p->r;
  d.h = p->H / p->r; d.w = p->W / p->r;
  d.bf16 = p->logit_dtype == MULO_BF16;
  d.invT = 1.0f / p->temperature;
  d.cfg_scale = p->cfg_scale;
  d.top_k = (p->top_k > 0 && p->top_k < p->V) ? p->top_k : 0;
  d.accept_mode = p->accept_mode;
  d.tau = (double)p->tau;
  d.pool_k = p->pool_k > 1 ? p->pool_k : 1;
  d.pool_delta = (double)p->pool_delta;
  d.radius = p->radius; d.clip = p->clip_before_first != 0; d.resample_mode = p->resample_mode;
  d.seed_lo = (uint32_t)(p->seed & 0xffffffffu); d.seed_hi = (uint32_t)(p->seed >> 32);
  d.round = p->round; d.image_offset = p->image_offset;
  return d;
}

static size_t pool_smem_bytes(const DevParams& d) {
  if (d.pool_k <= 1) return 0;
  return (size_t)d.pool_k * sizeof(double) + (size_t)((d.V + 31) / 32) * 4;
}

struct Workspace {
  uint32_t* status;
  uint8_t* flags;
  int32_t* cand_res;
  int32_t* cand_tgt;
  int32_t* fail_list;   // positions the streaming kernel leaves to the dense routines
  size_t bytes;
};

static Workspace carve_ws(void* base, const mulo_params* p) {
  const size_t n = (size_t)p->B * p->H * p->W;
  Workspace w;
  char* c = (char*)base;
  size_t off = 0;
  w.status = (uint32_t*)(c + off); off += kStatusBytes;
  w.flags = (uint8_t*)(c + off); off += align_up(n, 256);
  w.cand_res = (int32_t*)(c + off); off += align_up(n * 4, 256);
  w.cand_tgt = (int32_t*)(c + off); off += align_up(n * 4, 256);
  w.fail_list = (int32_t*)(c + off); off += align_up(n * 4, 256);
  w.bytes = off;
  return w;
}

extern "C" {

const char* mulo_status_string(mulo_status s) {
  switch (s) {
    case MULO_OK: return "ok";
    case MULO_ERR_INVALID_ARG: return "invalid argument";
    case MULO_ERR_UNSUPPORTED: return "unsupported size or parameter";
    case MULO_ERR_WORKSPACE: return "workspace missing or too small";
    case MULO_ERR_CUDA: return "CUDA runtime error";
    case MULO_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

mulo_status mulo_create(mulo_ctx** out, int device) {
  if (!out) return MULO_ERR_INVALID_ARG;
  *out = nullptr;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) {
    cudaGetLastError();
    return MULO_ERR_CUDA;
  }
  if (cudaSetDevice(device) != cudaSuccess) return MULO_ERR_CUDA;
  mulo_ctx* c = new (std::nothrow) mulo_ctx();
  if (!c) return MULO_ERR_INVALID_ARG;
  c->device = device;
  c->sm_count = prop.multiProcessorCount;
  c->smem_optin = (int)prop.sharedMemPerBlockOptin;
  c->ws = nullptr;
  c->ws_bytes = 0;
  c->launches = 0;
  c->ev_used = 0;
  c->force_dense = 0;
  c->no_lane = 0;
  *out = c;
  return MULO_OK;
}

void mulo_destroy(mulo_ctx* ctx) {
  if (!ctx) return;
  for (cudaEvent_t e : ctx->ev) cudaEventDestroy(e);
  delete ctx;
}

mulo_status mulo_set_general_path_only(mulo_ctx* ctx, int on) {
  if (!ctx) return MULO_ERR_INVALID_ARG;
  ctx->force_dense = on != 0;
  return MULO_OK;
}

mulo_status mulo_set_timing(mulo_ctx* ctx, int max_launches) {
  if (!ctx || max_launches < 0 || max_launches > 4096) return MULO_ERR_INVALID_ARG;
  for (cudaEvent_t e : ctx->ev) cudaEventDestroy(e);
  ctx->ev.clear();
  ctx->ev_used = 0;
  for (int i = 0; i < 2 * max_launches; ++i) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return MULO_ERR_CUDA;
    ctx->ev.push_back(e);
  }
  return MULO_OK;
}

mulo_status mulo_read_timing(mulo_ctx* ctx, double* row_kernel_ms, uint64_t* row_kernel_launches) {
  if (!ctx || !row_kernel_ms || !row_kernel_launches) return MULO_ERR_INVALID_ARG;
  double total = 0.0;
  for (size_t i = 0; i + 1 < ctx->ev_used; i += 2) {
    if (cudaEventSynchronize(ctx->ev[i + 1]) != cudaSuccess) return MULO_ERR_CUDA;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ctx->ev[i], ctx->ev[i + 1]) != cudaSuccess) return MULO_ERR_CUDA;
    total += ms;
  }
  *row_kernel_ms = total;
  *row_kernel_launches = ctx->ev_used / 2;
  ctx->ev_used = 0;
  return MULO_OK;
}

mulo_status mulo_workspace_bytes(const mulo_params* p, size_t* bytes) {
  mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  if (!bytes) return MULO_ERR_INVALID_ARG;
  *bytes = carve_ws(nullptr, p).bytes;
  return MULO_OK;
}

mulo_status mulo_set_workspace(mulo_ctx* ctx, void* dev_ptr, size_t bytes) {
  if (!ctx || !dev_ptr || ((uintptr_t)dev_ptr & 255u) || bytes < kStatusBytes) return MULO_ERR_INVALID_ARG;
  if (cudaMemset(dev_ptr, 0, kStatusBytes) != cudaSuccess) return MULO_ERR_CUDA;
  ctx->ws = dev_ptr;
  ctx->ws_bytes = bytes;
  return MULO_OK;
}

mulo_status mulo_status_of_device_flags(uint32_t flags) {
  return (flags & MULO_DEV_TIMEOUT) ? MULO_ERR_TIMEOUT : MULO_OK;
}

mulo_status mulo_poll_device_status(mulo_ctx* ctx, void* stream, uint32_t* flags) {
  if (!ctx || !flags) return MULO_ERR_INVALID_ARG;
  if (!ctx->ws) return MULO_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(flags, ctx->ws, sizeof(uint32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) return MULO_ERR_CUDA;
  if (cudaMemsetAsync(ctx->ws, 0, sizeof(uint32_t), st) != cudaSuccess) return MULO_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return MULO_ERR_CUDA;
  return mulo_status_of_device_flags(*flags);
}

mulo_status mulo_poll_fallback_counts(mulo_ctx* ctx, void* stream, uint32_t counts[5]) {
  if (!ctx || !counts) return MULO_ERR_INVALID_ARG;
  if (!ctx->ws) return MULO_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  char* src = (char*)ctx->ws + sizeof(uint32_t);
  if (cudaMemcpyAsync(counts, src, 5 * sizeof(uint32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) return MULO_ERR_CUDA;
  if (cudaMemsetAsync(src, 0, 5 * sizeof(uint32_t), st) != cudaSuccess) return MULO_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return MULO_ERR_CUDA;
  return MULO_OK;
}

mulo_status mulo_kernel_launches(const mulo_ctx* ctx, uint64_t* count) {
  if (!ctx || !count) return MULO_ERR_INVALID_ARG;
  *count = ctx->launches;
  return MULO_OK;
}

}  // extern "C"

static mulo_status check_ws(mulo_ctx* ctx, const mulo_params* p, Workspace* w) {
  if (!ctx->ws) return MULO_ERR_WORKSPACE;
  *w = carve_ws(ctx->ws, p);
  if (w->bytes > ctx->ws_bytes) return MULO_ERR_WORKSPACE;
  return MULO_OK;
}

static mulo_status launched(mulo_ctx* ctx, int n) {
  if (cudaGetLastError() != cudaSuccess) return MULO_ERR_CUDA;
  ctx->launches += (uint64_t)n;
  return MULO_OK;
}

template <class K>
static bool raise_smem(K kernel, size_t bytes, const mulo_ctx* ctx) {
  if (bytes + sizeof(BlockScratch) + 1024 > (size_t)ctx->smem_optin) return false;
  if (bytes > 0)
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) {
      cudaGetLastError();
      return false;
    }
  return true;
}


// ---- the fast top-k path of mulo_round -------------------------------------------------

// inverse of the standard normal CDF by bisection (host, set-up only)
static double inv_norm_cdf(double p) {
  double lo = -12.0, hi = 12.0;
  for (int i = 0; i < 200; ++i) {
    const double mid = 0.5 * (lo + hi);
    if (0.5 * erfc(-mid / sqrt(2.0)) < p) lo = mid; else hi = mid;
  }
  return 0.5 * (lo + hi);
}

// Fills `s` and returns the dynamic shared memory the streaming kernel needs, or 0 if these
// parameters are not eligible (then the general kernel runs).
static size_t plan_stream(const mulo_ctx* ctx, const DevParams& d, StreamArgs* s) {
  if (d.top_k <= 0) return 0;
  // pooling keeps a bitmap of the pooled token ids in the row's selection scratch (2 KB)
  if (d.pool_k > 1 && d.V > 16384) return 0;
  const int V = d.V, k = d.top_k;
  if (V < 1024 || 1 + d.r * d.r > kMaxRowsPerParent) return 0;
  // candidates aimed for beyond k: about six standard deviations of the count of entries
  // above a fixed value near the k-th largest
  const int margin = (int)fmax(64.0, 6.0 * sqrt((double)k));
  const int margin_boot = margin + 3 * margin / 4;   // rows without a prediction: the pivot comes from one chunk's statistics
  if ((double)(k + margin_boot) > 0.5 * V) return 0;
  const int esz = d.bf16 ? 2 : 4;
  const int epl = 16 / esz, piece = 32 * epl;
  s->chunk = kChunkPieces * piece;
  s->n_chunks = (V + s->chunk - 1) / s->chunk;
  if (s->n_chunks > 255) return 0;
  s->n_seg = s->n_chunks * kSWarps;
  // capacity of a row's candidate array: the bootstrap density's mean plus six standard
  // deviations of a binomial(V, density) count, rounded up to a multiple of 64
  const double pb = (double)(k + margin_boot) / V;
  int cap = (int)ceil(V * pb + 6.0 * sqrt(V * pb * (1.0 - pb)));
  cap += s->n_seg;              // every segment's run is rounded up to an even length
  {   // a segment of the draft row may hold at most 255 candidates (8-bit offsets in its look-up table)
    const double seg_mean = (double)kPPW * piece * pb;
    if (seg_mean + 6.0 * sqrt(seg_mean * (1.0 - pb)) > 255.0) return 0;
  }
  cap = (cap + 63) / 64 * 64;
  if (cap > 65535) return 0;
  s->cap = cap;
  s->margin = margin;
  s->a_theta = (float)inv_norm_cdf(1.0 - (double)k / V);
  s->a_boot = (float)inv_norm_cdf(1.0 - (double)(k + margin_boot) / V);
  const size_t dyn = stream_layout(*s, esz);
  const size_t fixed = sizeof(StreamSmem) + 1024;
  if (dyn + fixed > (size_t)ctx->smem_optin) return 0;
  return dyn;
}

template <bool BF16, bool HAS_U, bool SAMPLE = false, bool POOL = false>
static bool launch_stream_t(const mulo_ctx* ctx, const StreamArgs& s, size_t dyn, cudaStream_t st) {
  auto kern = k_round_stream<BF16, HAS_U, SAMPLE, POOL>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kSThreads, dyn) != cudaSuccess || per_sm < 1) {
    cudaGetLastError();
    return false;
  }
  int grid = ctx->sm_count * per_sm;
  if (grid > s.n_parents) grid = s.n_parents;
  kern<<<grid, kSThreads, dyn, st>>>(s);
  return true;
}

static bool launch_stream(const mulo_ctx* ctx, const StreamArgs& s, size_t dyn, cudaStream_t st) {
  const bool hu = s.uncond != nullptr;
  if (s.P.pool_k > 1) {
    if (s.P.bf16)
      return hu ? launch_stream_t<true, true, false, true>(ctx, s, dyn, st)
                : launch_stream_t<true, false, false, true>(ctx, s, dyn, st);
    return hu ? launch_stream_t<false, true, false, true>(ctx, s, dyn, st)
              : launch_stream_t<false, false, false, true>(ctx, s, dyn, st);
  }
  if (s.P.bf16) return hu ? launch_stream_t<true, true>(ctx, s, dyn, st) : launch_stream_t<true, false>(ctx, s, dyn, st);
  return hu ? launch_stream_t<false, true>(ctx, s, dyn, st) : launch_stream_t<false, false>(ctx, s, dyn, st);
}

// ---- the lane-private fast path (V = 256 * W, W <= 64) ---------------------------------

typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up once (host code only; no device work, no allocation).
static TensorMapEncodeFn tensor_map_encoder() {
  static std::once_flag once;
  static TensorMapEncodeFn fn = nullptr;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (TensorMapEncodeFn)p;
    else
      cudaGetLastError();
  });
  return fn;
}

// A logit tensor [rows, V] seen as [rows][256 threads][W ids]; one box = one phase of one warp's
// part of a row: the next 32 bytes of the id range of each of its 32 lanes, laid down with the
// 32-byte swizzle.
static bool encode_row_map(CUtensorMap* tm, const void* base, size_t rows, int V, bool bf16) {
  TensorMapEncodeFn enc = tensor_map_encoder();
  if (!enc || rows == 0 || rows > 0xffffffffull) return false;
  const int esz = bf16 ? 2 : 4, W = V / kLThreads;
  const cuuint64_t gdim[3] = {(cuuint64_t)W, (cuuint64_t)kLThreads, (cuuint64_t)rows};
  const cuuint64_t gstr[2] = {(cuuint64_t)W * esz, (cuuint64_t)V * esz};
  const cuuint32_t box[3] = {(cuuint32_t)(32 / esz), 32u, 1u};   // one warp's lanes
  const cuuint32_t es[3] = {1u, 1u, 1u};
  return enc(tm, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base),
             gdim, gstr, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_32B,
             CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Fills `s` and returns the dynamic shared memory the lane kernel needs, or 0 if these
// parameters are not eligible.
static size_t plan_lane(const mulo_ctx* ctx, const DevParams& d, LaneArgs* s) {
  if (d.top_k <= 0 || d.pool_k > 1) return 0;
  const int V = d.V, k = d.top_k;
  const int ids = d.bf16 ? 16 : 8;
  if (V % (kLThreads * ids) != 0 || V / kLThreads > 64) return 0;
  if (!tensor_map_encoder()) return 0;
  // candidates aimed for beyond k: six standard deviations of the count of entries above a fixed
  // value near the k-th largest (a row that comes up short is redone by the general routines, and
  // even one such row costs more than the margin does)
  const double p = (double)k / V;
  const int margin = (int)fmax(64.0, 6.0 * sqrt(k * (1.0 - p)));
  const int margin_boot = margin + 3 * margin / 4;   // rows without a prediction
  if ((double)(k + margin_boot) > 0.5 * V) return 0;
  // A list column serves two threads and holds four stacks (each thread's entries of the draft row
  // and of the current target row): the bootstrap density's mean for 4 W ids plus six and a half
  // standard deviations of that binomial count.  Three CTAs per SM are worth a somewhat shorter
  // column (five and a half deviations).
  const double pb = (double)(k + margin_boot) / V;
  const double mu = (double)(V / kLThreads) * pb, var = mu * (1.0 - pb);   // entries of one thread in one row
  const double quad_mean = 4.0 * mu, quad_sd = sqrt(4.0 * var);
  // ... and a thread stops appending when fewer rows than one phase's ids are left before the other
  // thread's stack, so the column must also hold both draft stacks, what the thread has gathered
  // by its last phase, and one more phase
  const int n_ph = (V / kLThreads) / ids;
  const double part = (double)(n_ph - 1) / n_ph;
  auto rows_needed = [&](double dev) {
    const double a1 = quad_mean + dev * quad_sd + 2.0;
    const double a2 = (2.0 + part) * mu + dev * sqrt(var * (2.0 + part * part)) + ids + 2.0;
    return (int)ceil(fmax(a1, a2));
  };
  int R = rows_needed(6.5);
  if (R < 16) R = 16;
  const size_t fixed = sizeof(LaneSmem) + 128 + 1024 + 256 + (size_t)kLRing;
  const size_t per_cta3 = (size_t)228 * 1024 / 3;
  if (per_cta3 > fixed) {
    const int R3 = (int)((per_cta3 - fixed) / 512);
    if (R3 < R && R3 >= rows_needed(5.5)) R = R3;
  }
  // one thread's own entries must fit the 32-bit mask of its low entries
  if (0.25 * quad_mean + 6.5 * sqrt(0.25 * quad_mean * (1.0 - pb)) > 32.0) return 0;
  const size_t dyn = 256 + (size_t)kLRing + (size_t)R * 512;
  if (dyn + sizeof(LaneSmem) + 128 + 1024 > (size_t)ctx->smem_optin) return 0;
  s->W = V / kLThreads;
  s->n_ph = s->W / ids;
  s->R = R;
  s->margin = margin;
  s->a_theta = (float)inv_norm_cdf(1.0 - p);
  s->a_boot = (float)inv_norm_cdf(1.0 - (double)(k + margin_boot) / V);
  s->a_max = (float)inv_norm_cdf(1.0 - 0.5 / V);
  return dyn;
}

// ---- rows without a top-k cut: the resident-row kernel ------------------------------------
// Eligible: top-k off, V = 256 * W with W a multiple of the ids in 16 bytes, and the rows of one
// position (draft row if q is needed, conditional, unconditional) within a CTA's shared memory.
static bool round_needs_q(const DevParams& d) {
  return !(d.accept_mode == MULO_ACCEPT_THRESHOLD && d.resample_mode == MULO_RESAMPLE_TARGET_ALL);
}

static size_t plan_full(const mulo_ctx* ctx, const DevParams& d, bool has_u, FullArgs* s) {
  if (d.top_k > 0 && d.top_k < d.V) return 0;
  const int esz = d.bf16 ? 2 : 4, n = 16 / esz;
  if (d.V % (kFThreads * n) != 0) return 0;
  const int need_q = round_needs_q(d) ? 1 : 0;
  const size_t rows = (size_t)need_q + 1 + (has_u ? 1 : 0);
  const size_t dyn = rows * (size_t)d.V * esz + (size_t)d.V / 8 + (size_t)kFThreads * 8;
  if (dyn + sizeof(FullSmem) + 1024 > (size_t)ctx->smem_optin) return 0;
  s->W = d.V / kFThreads;
  s->need_q = need_q;
  return dyn;
}

template <bool BF16, bool HAS_U>
static bool launch_full_t(const mulo_ctx* ctx, const FullArgs& s, size_t dyn, cudaStream_t st) {
  auto kern = k_round_full<BF16, HAS_U>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kFThreads, dyn) != cudaSuccess || per_sm < 1) {
    cudaGetLastError();
    return false;
  }
  int grid = ctx->sm_count * per_sm;
  if (grid > s.n_parents) grid = s.n_parents;
  kern<<<grid, kFThreads, dyn, st>>>(s);
  return true;
}

static bool launch_full(const mulo_ctx* ctx, const FullArgs& s, size_t dyn, cudaStream_t st) {
  const bool hu = s.uncond != nullptr;
  if (s.P.bf16) return hu ? launch_full_t<true, true>(ctx, s, dyn, st) : launch_full_t<true, false>(ctx, s, dyn, st);
  return hu ? launch_full_t<false, true>(ctx, s, dyn, st) : launch_full_t<false, false>(ctx, s, dyn, st);
}

template <bool BF16, bool HAS_U>
static bool launch_lane_t(const mulo_ctx* ctx, const LaneArgs& s, const CUtensorMap& tc, const CUtensorMap& tu,
                          const CUtensorMap& tq, size_t dyn, cudaStream_t st) {
  auto kern = k_round_lane<BF16, HAS_U>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kLThreads, dyn) != cudaSuccess || per_sm < 1) {
    cudaGetLastError();
    return false;
  }
  int grid = ctx->sm_count * per_sm;
  if (grid > s.n_parents) grid = s.n_parents;
  kern<<<grid, kLThreads, dyn, st>>>(s, tc, tu, tq);
  return true;
}

static bool launch_lane(const mulo_ctx* ctx, const LaneArgs& s, size_t dyn, cudaStream_t st) {
  const DevParams& d = s.P;
  CUtensorMap tc, tu, tq;
  const size_t rows = (size_t)d.B * d.H * d.W, cells = (size_t)d.B * d.h * d.w;
  if (!encode_row_map(&tc, s.cond, rows, d.V, d.bf16)) return false;
  if (!encode_row_map(&tu, s.uncond ? s.uncond : s.cond, rows, d.V, d.bf16)) return false;
  if (!encode_row_map(&tq, s.draft, cells, d.V, d.bf16)) return false;
  const bool hu = s.uncond != nullptr;
  if (d.bf16) return hu ? launch_lane_t<true, true>(ctx, s, tc, tu, tq, dyn, st) : launch_lane_t<true, false>(ctx, s, tc, tu, tq, dyn, st);
  return hu ? launch_lane_t<false, true>(ctx, s, tc, tu, tq, dyn, st) : launch_lane_t<false, false>(ctx, s, tc, tu, tq, dyn, st);
}

static size_t mask_smem(const mulo_params* p) { return (size_t)3 * p->H * ((p->W + 31) / 32) * 4; }

// Everything mulo_round can refuse without touching the device.
static mulo_status check_round_args(const mulo_ctx* ctx, const mulo_params* p, const void* tgt_cond,
                                    const void* tgt_uncond, const void* draft_logits_lo, const int32_t* draft_tok_lo,
                                    const uint16_t* nn, const int32_t* out_tok, const uint32_t* reject_bits,
                                    const uint32_t* expand_bits) {
  if (!ctx) return MULO_ERR_INVALID_ARG;
  mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  if (!tgt_cond || !draft_logits_lo || !draft_tok_lo || !out_tok || !reject_bits || !expand_bits)
    return MULO_ERR_INVALID_ARG;
  if (p->pool_k > 1 && !nn) return MULO_ERR_INVALID_ARG;
  if (!aligned16(tgt_cond) || !aligned16(tgt_uncond) || !aligned16(draft_logits_lo)) return MULO_ERR_INVALID_ARG;
  return on_context_device(ctx);
}

extern "C" {

mulo_status mulo_upsample_pool(mulo_ctx* ctx, const mulo_params* p, const void* draft_logits_lo,
                               const int32_t* draft_tok_lo, const uint16_t* nn, int32_t* draft_tok_hi,
                               float* draft_stats_lo, float* q_tok_hi, void* stream) {
  (void)nn;
  if (!ctx) return MULO_ERR_INVALID_ARG;
  mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  if (!draft_logits_lo || !draft_tok_lo || !draft_tok_hi || !draft_stats_lo || !q_tok_hi) return MULO_ERR_INVALID_ARG;
  if (!aligned16(draft_logits_lo)) return MULO_ERR_INVALID_ARG;
  if (!ctx->ws) return MULO_ERR_WORKSPACE;
  if (p->B == 0) return MULO_OK;
  if ((s = on_context_device(ctx)) != MULO_OK) return s;
  RowKernelArgs a;
  memset(&a, 0, sizeof a);
  a.P = to_dev(p);
  a.draft = (const char*)draft_logits_lo;
  a.draft_tok_lo = draft_tok_lo;
  a.tok_hi_out = draft_tok_hi;
  a.stats_out = draft_stats_lo;
  a.q_tok_hi_out = q_tok_hi;
  a.dev_status = (uint32_t*)ctx->ws;
  k_upsample_pool<<<p->B * a.P.h * a.P.w, kThreads, 0, (cudaStream_t)stream>>>(a);
  return launched(ctx, 1);
}

mulo_status mulo_island_schedule(mulo_ctx* ctx, const mulo_params* p, const int32_t* labels, int32_t window,
                                 int32_t* step, int32_t* n_steps, void* stream) {
  if (!ctx) return MULO_ERR_INVALID_ARG;
  mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  if (!labels || !step || !n_steps || window < 1) return MULO_ERR_INVALID_ARG;
  if ((size_t)p->H * p->W > (size_t)kIslandMaxCells) return MULO_ERR_UNSUPPORTED;
  if (p->B == 0) return MULO_OK;
  if ((s = on_context_device(ctx)) != MULO_OK) return s;
  ScheduleArgs a;
  a.H = p->H; a.W = p->W; a.window = window > p->W ? p->W : window;
  a.labels = labels; a.step = step; a.n_steps = n_steps;
  const size_t smem = (size_t)4 * p->W * sizeof(int);
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(k_island_schedule, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    cudaGetLastError();
    return MULO_ERR_CUDA;
  }
  k_island_schedule<<<p->B, kScheduleThreads, smem, (cudaStream_t)stream>>>(a);
  return launched(ctx, 1);
}

mulo_status mulo_redraw_plan(mulo_ctx* ctx, const mulo_params* p, const int32_t* step, int32_t max_step,
                             int32_t* pos_list, int32_t* step_offsets, void* stream) {
  if (!ctx) return MULO_ERR_INVALID_ARG;
  mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  if (!step || !pos_list || !step_offsets || max_step < 1) return MULO_ERR_INVALID_ARG;
  if ((size_t)max_step > (size_t)p->H * p->W) return MULO_ERR_INVALID_ARG;
  if ((s = on_context_device(ctx)) != MULO_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  const int n = p->B * p->H * p->W;
  int32_t* cursor = step_offsets + max_step + 2;
  if (cudaMemsetAsync(step_offsets, 0, sizeof(int32_t) * 2 * ((size_t)max_step + 2), st) != cudaSuccess) return MULO_ERR_CUDA;
  if (n == 0) return MULO_OK;
  const int blocks = (n + 255) / 256 < 4 * ctx->sm_count ? (n + 255) / 256 : 4 * ctx->sm_count;
  k_redraw_count<<<blocks, 256, 0, st>>>(step, n, max_step, cursor);
  k_redraw_scan<<<1, kScanThreads, 0, st>>>(max_step, step_offsets, cursor);
  k_redraw_fill<<<blocks, 256, 0, st>>>(step, n, max_step, cursor, pos_list);
  return launched(ctx, 3);
}

mulo_status mulo_redraw_step(mulo_ctx* ctx, const mulo_params* p, int32_t s_index, int32_t max_step,
                             const int32_t* pos_list, const int32_t* step_offsets, const void* tgt_cond,
                             const void* tgt_uncond, int32_t* out_tok, void* stream) {
  if (!ctx) return MULO_ERR_INVALID_ARG;
  mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  if (!pos_list || !step_offsets || !tgt_cond || !out_tok || !aligned16(tgt_cond) || !aligned16(tgt_uncond))
    return MULO_ERR_INVALID_ARG;
  if (s_index < 1 || s_index > max_step) return MULO_ERR_INVALID_ARG;
  if (p->B == 0) return MULO_OK;
  if ((s = on_context_device(ctx)) != MULO_OK) return s;
  RedrawArgs a;
  memset(&a, 0, sizeof a);
  a.P = to_dev(p);
  a.cond = (const char*)tgt_cond;
  a.uncond = (const char*)tgt_uncond;
  a.pos_list = pos_list;
  a.offsets = step_offsets;
  a.out_tok = out_tok;
  a.s = s_index;
  // the step's positions are counted on the device: a fixed grid strides over them
  k_redraw_step<<<2 * ctx->sm_count, kThreads, 0, (cudaStream_t)stream>>>(a);
  return launched(ctx, 1);
}

mulo_status mulo_sample_draft(mulo_ctx* ctx, const mulo_params* p, const void* draft_logits_lo,
                              int32_t* draft_tok_lo, void* stream) {
  if (!ctx) return MULO_ERR_INVALID_ARG;
  mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  if (!draft_logits_lo || !draft_tok_lo || !aligned16(draft_logits_lo)) return MULO_ERR_INVALID_ARG;
  if (!ctx->ws) return MULO_ERR_WORKSPACE;
  if (p->B == 0) return MULO_OK;
  if ((s = on_context_device(ctx)) != MULO_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  RowKernelArgs a;
  memset(&a, 0, sizeof a);
  a.P = to_dev(p);
  a.draft = (const char*)draft_logits_lo;
  a.out_tok = draft_tok_lo;
  a.dev_status = (uint32_t*)ctx->ws;
  // fast path: the streaming kernel in its sampling mode (top-k on, and a workspace large
  // enough for the list of cells it may leave to the general routines)
  Workspace w;
  StreamArgs sa;
  memset(&sa, 0, sizeof sa);
  const size_t sdyn = (ctx->force_dense || check_ws(ctx, p, &w) != MULO_OK) ? 0 : plan_stream(ctx, a.P, &sa);
  if (sdyn) {
    sa.P = a.P;
    sa.draft = a.draft;
    sa.sample_out = draft_tok_lo;
    sa.dev_status = w.status;
    sa.fail_list = w.fail_list;
    sa.n_parents = p->B * a.P.h * a.P.w;
    if (cudaMemsetAsync(w.status + kFailCount, 0, sizeof(uint32_t), st) != cudaSuccess) return MULO_ERR_CUDA;
    const bool fast = a.P.bf16 ? launch_stream_t<true, false, true>(ctx, sa, sdyn, st)
                               : launch_stream_t<false, false, true>(ctx, sa, sdyn, st);
    if (fast) {
      k_sample_failed<<<2 * ctx->sm_count, kThreads, 0, st>>>(a, w.fail_list, w.status + kFailCount);
      return launched(ctx, 2);
    }
  }
  k_sample_draft<<<p->B * a.P.h * a.P.w, kThreads, 0, st>>>(a);
  return launched(ctx, 1);
}

mulo_status mulo_downsample(mulo_ctx* ctx, const mulo_params* p, const int32_t* tok_hi, int32_t* tok_lo,
                            void* stream) {
  if (!ctx) return MULO_ERR_INVALID_ARG;
  mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  if (!tok_hi || !tok_lo) return MULO_ERR_INVALID_ARG;
  if (p->r > 16) return MULO_ERR_UNSUPPORTED;
  if (p->B == 0) return MULO_OK;
  if ((s = on_context_device(ctx)) != MULO_OK) return s;
  const int h = p->H / p->r, w = p->W / p->r, cells = p->B * h * w;
  k_downsample<<<(cells + 255) / 256, 256, 0, (cudaStream_t)stream>>>(tok_hi, tok_lo, cells, h, w, p->W, p->r);
  return launched(ctx, 1);
}

mulo_status mulo_verify(mulo_ctx* ctx, const mulo_params* p, const void* tgt_cond, const void* tgt_uncond,
                        const void* draft_logits_lo, const float* draft_stats_lo,
                        const int32_t* draft_tok_hi, const uint16_t* nn, float* p_tok, float* q_tok,
                        float* accept_prob, uint32_t* reject_bits, int32_t* n_reject,
                        int32_t* first_reject, void* stream) {
  if (!ctx) return MULO_ERR_INVALID_ARG;
  mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  if (!tgt_cond || !draft_logits_lo || !draft_stats_lo || !draft_tok_hi || !p_tok || !q_tok || !accept_prob ||
      !reject_bits || !n_reject || !first_reject)
    return MULO_ERR_INVALID_ARG;
  if (p->pool_k > 1 && !nn) return MULO_ERR_INVALID_ARG;
  if (!aligned16(tgt_cond) || !aligned16(tgt_uncond) || !aligned16(draft_logits_lo)) return MULO_ERR_INVALID_ARG;
  Workspace w;
  if ((s = check_ws(ctx, p, &w)) != MULO_OK) return s;
  if (p->B == 0) return MULO_OK;
  if ((s = on_context_device(ctx)) != MULO_OK) return s;
  RowKernelArgs a;
  memset(&a, 0, sizeof a);
  a.P = to_dev(p);
  a.cond = (const char*)tgt_cond;
  a.uncond = (const char*)tgt_uncond;
  a.draft = (const char*)draft_logits_lo;
  a.stats_in = draft_stats_lo;
  a.draft_tok_hi = draft_tok_hi;
  a.nn = nn;
  a.p_tok = p_tok; a.q_tok = q_tok; a.accept_prob = accept_prob;
  a.flags = w.flags;
  a.dev_status = w.status;
  const size_t dyn = pool_smem_bytes(a.P);
  if (!raise_smem(k_verify_rows<false>, dyn, ctx)) return MULO_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  k_verify_rows<false><<<(unsigned)((size_t)p->B * p->H * p->W), kThreads, dyn, st>>>(a);
  MaskArgs m;
  memset(&m, 0, sizeof m);
  m.H = p->H; m.W = p->W; m.r = p->r; m.radius = p->radius; m.clip = a.P.clip; m.resample_mode = p->resample_mode;
  m.flags = w.flags;
  m.reject_bits = reject_bits; m.n_reject = n_reject; m.first_reject = first_reject;
  k_mask<0><<<p->B, kMaskThreads, mask_smem(p), st>>>(m);
  return launched(ctx, 2);
}

mulo_status mulo_local_reject_expand(mulo_ctx* ctx, const mulo_params* p, const uint32_t* reject_bits,
                                     const int32_t* first_reject, uint32_t* expand_bits,
                                     int32_t* n_expand, void* stream) {
  if (!ctx) return MULO_ERR_INVALID_ARG;
  mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  if (!reject_bits || !first_reject || !expand_bits || !n_expand) return MULO_ERR_INVALID_ARG;
  if (p->B == 0) return MULO_OK;
  if ((s = on_context_device(ctx)) != MULO_OK) return s;
  MaskArgs m;
  memset(&m, 0, sizeof m);
  m.H = p->H; m.W = p->W; m.r = p->r; m.radius = p->radius; m.clip = p->clip_before_first != 0;
  m.resample_mode = p->resample_mode;
  m.reject_in = reject_bits; m.first_in = first_reject;
  m.expand_bits = expand_bits; m.n_expand = n_expand;
  k_mask<1><<<p->B, kMaskThreads, mask_smem(p), (cudaStream_t)stream>>>(m);
  return launched(ctx, 1);
}

mulo_status mulo_islands(mulo_ctx* ctx, const mulo_params* p, const uint32_t* expand_bits, int32_t* labels,
                         int32_t* n_islands, int32_t max_islands, int32_t* island_rows,
                         int32_t* island_size, void* stream) {
  if (!ctx) return MULO_ERR_INVALID_ARG;
  mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  if (!expand_bits || !labels || !n_islands || max_islands < 0) return MULO_ERR_INVALID_ARG;
  if ((size_t)p->H * p->W > (size_t)kIslandMaxCells) return MULO_ERR_UNSUPPORTED;
  if (p->B == 0) return MULO_OK;
  if ((s = on_context_device(ctx)) != MULO_OK) return s;
  IslandArgs a;
  a.H = p->H; a.W = p->W; a.max_islands = max_islands;
  a.bits = expand_bits; a.labels = labels; a.n_islands = n_islands;
  a.rows = max_islands > 0 ? island_rows : nullptr;
  a.size = max_islands > 0 ? island_size : nullptr;
  const size_t smem = ((size_t)2 * p->H * p->W + (size_t)p->H * ((p->W + 31) / 32)) * sizeof(int);
  if (smem + 1024 > (size_t)ctx->smem_optin) return MULO_ERR_UNSUPPORTED;
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(k_islands, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    cudaGetLastError();
    return MULO_ERR_CUDA;
  }
  k_islands<<<p->B, kIslandThreads, smem, (cudaStream_t)stream>>>(a);
  return launched(ctx, 1);
}

mulo_status mulo_resample(mulo_ctx* ctx, const mulo_params* p, const void* tgt_cond, const void* tgt_uncond,
                          const void* draft_logits_lo, const float* draft_stats_lo,
                          const int32_t* draft_tok_hi, const uint16_t* nn, const uint32_t* reject_bits,
                          const uint32_t* expand_bits, int32_t* out_tok, void* stream) {
  if (!ctx) return MULO_ERR_INVALID_ARG;
  mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  if (!tgt_cond || !draft_logits_lo || !draft_stats_lo || !draft_tok_hi || !reject_bits || !expand_bits || !out_tok)
    return MULO_ERR_INVALID_ARG;
  if (p->pool_k > 1 && !nn) return MULO_ERR_INVALID_ARG;
  if (!aligned16(tgt_cond) || !aligned16(tgt_uncond) || !aligned16(draft_logits_lo)) return MULO_ERR_INVALID_ARG;
  if (!ctx->ws) return MULO_ERR_WORKSPACE;
  if (p->B == 0) return MULO_OK;
  if ((s = on_context_device(ctx)) != MULO_OK) return s;
  RowKernelArgs a;
  memset(&a, 0, sizeof a);
  a.P = to_dev(p);
  a.cond = (const char*)tgt_cond;
  a.uncond = (const char*)tgt_uncond;
  a.draft = (const char*)draft_logits_lo;
  a.stats_in = draft_stats_lo;
  a.draft_tok_hi = draft_tok_hi;
  a.nn = nn;
  a.reject_bits = reject_bits;
  a.expand_bits = expand_bits;
  a.out_tok = out_tok;
  a.dev_status = (uint32_t*)ctx->ws;
  const size_t dyn = pool_smem_bytes(a.P);
  if (!raise_smem(k_resample_rows, dyn, ctx)) return MULO_ERR_UNSUPPORTED;
  k_resample_rows<<<(unsigned)((size_t)p->B * p->H * p->W), kThreads, dyn, (cudaStream_t)stream>>>(a);
  return launched(ctx, 1);
}

mulo_status mulo_round(mulo_ctx* ctx, const mulo_params* p, const void* tgt_cond, const void* tgt_uncond,
                       const void* draft_logits_lo, const int32_t* draft_tok_lo, const uint16_t* nn,
                       int32_t* out_tok, uint32_t* reject_bits, uint32_t* expand_bits, float* p_tok,
                       float* q_tok, float* accept_prob, int32_t* n_reject, int32_t* n_expand,
                       int32_t* first_reject, void* stream) {
  mulo_status s = check_round_args(ctx, p, tgt_cond, tgt_uncond, draft_logits_lo, draft_tok_lo, nn, out_tok,
                                   reject_bits, expand_bits);
  if (s != MULO_OK) return s;
  Workspace w;
  if ((s = check_ws(ctx, p, &w)) != MULO_OK) return s;
  if (p->B == 0) return MULO_OK;
  RowKernelArgs a;
  memset(&a, 0, sizeof a);
  a.P = to_dev(p);
  a.cond = (const char*)tgt_cond;
  a.uncond = (const char*)tgt_uncond;
  a.draft = (const char*)draft_logits_lo;
  a.draft_tok_lo = draft_tok_lo;
  a.nn = nn;
  a.p_tok = p_tok; a.q_tok = q_tok; a.accept_prob = accept_prob;
  a.flags = w.flags; a.cand_res = w.cand_res; a.cand_tgt = w.cand_tgt;
  a.dev_status = w.status;
  const size_t dyn = pool_smem_bytes(a.P);
  if (!raise_smem(k_verify_rows<true>, dyn, ctx)) return MULO_ERR_UNSUPPORTED;
  if (!raise_smem(k_verify_failed, dyn, ctx)) return MULO_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  const bool timed = ctx->ev_used + 2 <= ctx->ev.size();
  if (timed) cudaEventRecord(ctx->ev[ctx->ev_used], st);
  bool fast = false;
  int fast_launches = 2;   // a fast kernel and the one that redoes the rows it left
  // Eq. 5 with every redraw from the target distribution never looks at q: no kernel reports it
  // (the resident-row kernel does not even read the draft logits), the output is zero-filled
  if (!round_needs_q(a.P) && q_tok) {
    if (cudaMemsetAsync(q_tok, 0, sizeof(float) * (size_t)p->B * p->H * p->W, st) != cudaSuccess) return MULO_ERR_CUDA;
    a.q_tok = nullptr;
    q_tok = nullptr;
  }
  FullArgs fa;
  memset(&fa, 0, sizeof fa);
  const size_t fdyn = ctx->force_dense ? 0 : plan_full(ctx, a.P, tgt_uncond != nullptr, &fa);
  if (fdyn) {
    fa.P = a.P;
    fa.cond = a.cond; fa.uncond = a.uncond; fa.draft = a.draft; fa.draft_tok_lo = draft_tok_lo;
    fa.nn = a.nn;
    fa.p_tok = p_tok; fa.q_tok = q_tok; fa.accept_prob = accept_prob;
    fa.flags = w.flags; fa.cand_res = w.cand_res; fa.cand_tgt = w.cand_tgt;
    fa.dev_status = w.status;
    fa.n_parents = p->B * a.P.h * a.P.w;
    fast = launch_full(ctx, fa, fdyn, st);
    if (fast) fast_launches = 1;
  }
  LaneArgs la;
  memset(&la, 0, sizeof la);
  const size_t ldyn = (ctx->force_dense || ctx->no_lane || fast) ? 0 : plan_lane(ctx, a.P, &la);
  if (ldyn) {
    la.P = a.P;
    la.cond = a.cond; la.uncond = a.uncond; la.draft = a.draft; la.draft_tok_lo = draft_tok_lo;
    la.p_tok = p_tok; la.q_tok = q_tok; la.accept_prob = accept_prob;
    la.flags = w.flags; la.cand_res = w.cand_res; la.cand_tgt = w.cand_tgt;
    la.dev_status = w.status;
    la.fail_list = w.fail_list;
    la.n_parents = p->B * a.P.h * a.P.w;
    if (cudaMemsetAsync(w.status + kFailCount, 0, sizeof(uint32_t), st) != cudaSuccess) return MULO_ERR_CUDA;
    fast = launch_lane(ctx, la, ldyn, st);
    if (fast) k_verify_failed<<<2 * ctx->sm_count, kThreads, dyn, st>>>(a, w.fail_list, w.status + kFailCount);
  }
  StreamArgs sa;
  memset(&sa, 0, sizeof sa);
  const size_t sdyn = (ctx->force_dense || fast) ? 0 : plan_stream(ctx, a.P, &sa);
  if (sdyn) {
    sa.P = a.P;
    sa.cond = a.cond; sa.uncond = a.uncond; sa.draft = a.draft; sa.draft_tok_lo = draft_tok_lo;
    sa.nn = a.nn;
    sa.p_tok = p_tok; sa.q_tok = q_tok; sa.accept_prob = accept_prob;
    sa.flags = w.flags; sa.cand_res = w.cand_res; sa.cand_tgt = w.cand_tgt;
    sa.dev_status = w.status;
    sa.fail_list = w.fail_list;
    sa.n_parents = p->B * a.P.h * a.P.w;
    if (cudaMemsetAsync(w.status + kFailCount, 0, sizeof(uint32_t), st) != cudaSuccess) return MULO_ERR_CUDA;
    fast = launch_stream(ctx, sa, sdyn, st);
    // the rows the streaming kernel gave up on (usually a handful, often none)
    if (fast) k_verify_failed<<<2 * ctx->sm_count, kThreads, dyn, st>>>(a, w.fail_list, w.status + kFailCount);
  }
  if (!fast) k_verify_rows<true><<<p->B * a.P.h * a.P.w, kThreads, dyn, st>>>(a);
  if (timed) {
    cudaEventRecord(ctx->ev[ctx->ev_used + 1], st);
    ctx->ev_used += 2;
  }
  MaskArgs m;
  memset(&m, 0, sizeof m);
  m.H = p->H; m.W = p->W; m.r = p->r; m.radius = p->radius; m.clip = a.P.clip; m.resample_mode = p->resample_mode;
  m.flags = w.flags;
  m.reject_bits = reject_bits; m.expand_bits = expand_bits;
  m.n_reject = n_reject; m.first_reject = first_reject; m.n_expand = n_expand;
  m.cand_res = w.cand_res; m.cand_tgt = w.cand_tgt;
  m.draft_tok_lo = draft_tok_lo; m.out_tok = out_tok;
  k_mask<2><<<p->B, kMaskThreads, mask_smem(p), st>>>(m);
  return launched(ctx, fast ? 1 + fast_launches : 2);
}

mulo_status mulo_round_kernel(const mulo_ctx* ctx, const mulo_params* p, int has_uncond, int* kernel) {
  if (!ctx || !kernel) return MULO_ERR_INVALID_ARG;
  const mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  const DevParams d = to_dev(p);
  LaneArgs la;
  StreamArgs sa;
  memset(&la, 0, sizeof la);
  memset(&sa, 0, sizeof sa);
  *kernel = MULO_KERNEL_GENERAL;
  if (ctx->force_dense) return MULO_OK;
  FullArgs fa;
  memset(&fa, 0, sizeof fa);
  if (plan_full(ctx, d, has_uncond != 0, &fa)) *kernel = MULO_KERNEL_FULL;
  else if (!ctx->no_lane && plan_lane(ctx, d, &la)) *kernel = MULO_KERNEL_LANE;
  else if (plan_stream(ctx, d, &sa)) *kernel = MULO_KERNEL_STREAM;
  return MULO_OK;
}

// ---- host-buffer variant -------------------------------------------------------------

struct HostArena {
  size_t ws, cond, uncond, draft, tok_lo, nn, out_tok, rbits, ebits, ptok, qtok, aprob, nrej, nexp, first, total;
};

static HostArena carve_arena(const mulo_params* p, int has_uncond) {
  const size_t n = (size_t)p->B * p->H * p->W, nlo = n / ((size_t)p->r * p->r);
  const size_t esz = p->logit_dtype == MULO_BF16 ? 2 : 4;
  const size_t nwords = (size_t)p->B * p->H * ((p->W + 31) / 32);
  HostArena a;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes ? bytes : 1, 256); return o; };
  a.ws = take(carve_ws(nullptr, p).bytes);
  a.cond = take(n * p->V * esz);
  a.uncond = take(has_uncond ? n * p->V * esz : 0);
  a.draft = take(nlo * p->V * esz);
  a.tok_lo = take(nlo * 4);
  a.nn = take(p->pool_k > 1 ? (size_t)p->V * p->pool_k * 2 : 0);
  a.out_tok = take(n * 4);
  a.rbits = take(nwords * 4);
  a.ebits = take(nwords * 4);
  a.ptok = take(n * 4); a.qtok = take(n * 4); a.aprob = take(n * 4);
  a.nrej = take((size_t)p->B * 4); a.nexp = take((size_t)p->B * 4); a.first = take((size_t)p->B * 4);
  a.total = off;
  return a;
}

mulo_status mulo_round_host_arena_bytes(const mulo_params* p, int has_uncond, size_t* bytes) {
  mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  if (!bytes) return MULO_ERR_INVALID_ARG;
  *bytes = carve_arena(p, has_uncond).total;
  return MULO_OK;
}

mulo_status mulo_round_host(mulo_ctx* ctx, const mulo_params* p, void* arena, size_t arena_bytes,
                            const void* tgt_cond, const void* tgt_uncond, const void* draft_logits_lo,
                            const int32_t* draft_tok_lo, const uint16_t* nn, int32_t* out_tok,
                            uint32_t* reject_bits, uint32_t* expand_bits, float* p_tok, float* q_tok,
                            float* accept_prob, int32_t* n_reject, int32_t* n_expand,
                            int32_t* first_reject, void* stream) {
  if (!ctx || !arena || ((uintptr_t)arena & 255u)) return MULO_ERR_INVALID_ARG;
  mulo_status s = validate(p);
  if (s != MULO_OK) return s;
  if (!tgt_cond || !draft_logits_lo || !draft_tok_lo || !out_tok || !reject_bits || !expand_bits)
    return MULO_ERR_INVALID_ARG;
  if (p->pool_k > 1 && !nn) return MULO_ERR_INVALID_ARG;
  const HostArena A = carve_arena(p, tgt_uncond != nullptr);
  if (A.total > arena_bytes) return MULO_ERR_WORKSPACE;
  if (p->B == 0) return MULO_OK;
  if ((s = on_context_device(ctx)) != MULO_OK) return s;
  char* d = (char*)arena;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t n = (size_t)p->B * p->H * p->W, nlo = n / ((size_t)p->r * p->r);
  const size_t esz = p->logit_dtype == MULO_BF16 ? 2 : 4;
  const size_t nwords = (size_t)p->B * p->H * ((p->W + 31) / 32);
  bool ok = true;
  ok &= cudaMemsetAsync(d + A.ws, 0, kStatusBytes, st) == cudaSuccess;
  ctx->ws = d + A.ws;
  ctx->ws_bytes = carve_ws(nullptr, p).bytes;
  ok &= cudaMemcpyAsync(d + A.draft, draft_logits_lo, nlo * p->V * esz, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok &= cudaMemcpyAsync(d + A.tok_lo, draft_tok_lo, nlo * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (p->pool_k > 1)
    ok &= cudaMemcpyAsync(d + A.nn, nn, (size_t)p->V * p->pool_k * 2, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok &= cudaMemcpyAsync(d + A.cond, tgt_cond, n * p->V * esz, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (tgt_uncond)
    ok &= cudaMemcpyAsync(d + A.uncond, tgt_uncond, n * p->V * esz, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (!ok) return MULO_ERR_CUDA;
  s = mulo_round(ctx, p, d + A.cond, tgt_uncond ? d + A.uncond : nullptr, d + A.draft,
                 (const int32_t*)(d + A.tok_lo), p->pool_k > 1 ? (const uint16_t*)(d + A.nn) : nullptr,
                 (int32_t*)(d + A.out_tok), (uint32_t*)(d + A.rbits), (uint32_t*)(d + A.ebits),
                 p_tok ? (float*)(d + A.ptok) : nullptr, q_tok ? (float*)(d + A.qtok) : nullptr,
                 accept_prob ? (float*)(d + A.aprob) : nullptr, (int32_t*)(d + A.nrej),
                 (int32_t*)(d + A.nexp), (int32_t*)(d + A.first), stream);
  if (s != MULO_OK) return s;
  ok &= cudaMemcpyAsync(out_tok, d + A.out_tok, n * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  ok &= cudaMemcpyAsync(reject_bits, d + A.rbits, nwords * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  ok &= cudaMemcpyAsync(expand_bits, d + A.ebits, nwords * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (p_tok) ok &= cudaMemcpyAsync(p_tok, d + A.ptok, n * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (q_tok) ok &= cudaMemcpyAsync(q_tok, d + A.qtok, n * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (accept_prob) ok &= cudaMemcpyAsync(accept_prob, d + A.aprob, n * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (n_reject) ok &= cudaMemcpyAsync(n_reject, d + A.nrej, (size_t)p->B * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (n_expand) ok &= cudaMemcpyAsync(n_expand, d + A.nexp, (size_t)p->B * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (first_reject) ok &= cudaMemcpyAsync(first_reject, d + A.first, (size_t)p->B * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  ok &= cudaStreamSynchronize(st) == cudaSuccess;
  return ok ? MULO_OK : MULO_ERR_CUDA;
}

}  // extern "C"

// ---- allocation-free variant of the fused round ------------------------------------------

// Scratch of mulo_round_static: lives in the library image, one copy per device that
// loads it.  In host code this name is only a handle for the runtime's symbol table,
// never a device address; the kernels get the address cudaGetSymbolAddress returns.
static __device__ __align__(256) unsigned char g_static_scratch[MULO_STATIC_SCRATCH_BYTES];

static const int kMaxStaticDevices = 64;
static void* g_static_scratch_addr[kMaxStaticDevices];   // per device, nullptr until looked up
static std::mutex g_static_scratch_mutex;

// Device address of g_static_scratch on `device`: looked up once per device, with that
// device current, then served from the table.
static mulo_status static_scratch_address(int device, void** out) {
  if (device < 0 || device >= kMaxStaticDevices) return MULO_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (!g_static_scratch_addr[device]) {
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return MULO_ERR_CUDA;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) return MULO_ERR_CUDA;
    void* addr = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&addr, g_static_scratch);
    if (prev != device) cudaSetDevice(prev);
    if (e != cudaSuccess || !addr) {
      cudaGetLastError();
      return MULO_ERR_CUDA;
    }
    g_static_scratch_addr[device] = addr;
  }
  *out = g_static_scratch_addr[device];
  return MULO_OK;
}

extern "C" mulo_status mulo_round_static(mulo_ctx* ctx, const mulo_params* p, const void* tgt_cond,
                                         const void* tgt_uncond, const void* draft_logits_lo,
                                         const int32_t* draft_tok_lo, const uint16_t* nn, int32_t* out_tok,
                                         uint32_t* reject_bits, uint32_t* expand_bits, float* p_tok,
                                         float* q_tok, float* accept_prob, int32_t* n_reject,
                                         int32_t* n_expand, int32_t* first_reject, uint32_t* device_status,
                                         void* stream) {
  // every refusal comes before the shared array is touched
  mulo_status s = check_round_args(ctx, p, tgt_cond, tgt_uncond, draft_logits_lo, draft_tok_lo, nn, out_tok,
                                   reject_bits, expand_bits);
  if (s != MULO_OK) return s;
  if (carve_ws(nullptr, p).bytes > (size_t)MULO_STATIC_SCRATCH_BYTES) return MULO_ERR_WORKSPACE;
  void* scratch = nullptr;
  if ((s = static_scratch_address(ctx->device, &scratch)) != MULO_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  // The status word is OR-ed into and must start at zero; flags and candidates are written
  // for every position of this call before the mask kernel reads them.
  if (cudaMemsetAsync(scratch, 0, kStatusBytes, st) != cudaSuccess) return MULO_ERR_CUDA;
  void* const saved_ws = ctx->ws;
  const size_t saved_bytes = ctx->ws_bytes;
  ctx->ws = scratch;
  ctx->ws_bytes = MULO_STATIC_SCRATCH_BYTES;
  s = mulo_round(ctx, p, tgt_cond, tgt_uncond, draft_logits_lo, draft_tok_lo, nn, out_tok, reject_bits,
                 expand_bits, p_tok, q_tok, accept_prob, n_reject, n_expand, first_reject, stream);
  ctx->ws = saved_ws;
  ctx->ws_bytes = saved_bytes;
  if (s != MULO_OK) return s;
  if (device_status &&
      cudaMemcpyAsync(device_status, scratch, sizeof(uint32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return MULO_ERR_CUDA;
  return MULO_OK;
}
