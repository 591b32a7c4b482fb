// The fast path of the fused round for rows with top-k on (no pooling):
// a persistent CTA streams every logit row ONCE through a shared-memory ring
// filled by bulk-async copies (cp.async.bulk + mbarrier), keeps only the
// entries above a predicted pivot (a few hundred more than k), finds the exact
// k-th largest among them, and does softmax / acceptance / residual / inverse
// CDF on that short list.  A row whose prediction fails (too few or too many
// candidates) is redone by the dense routines from global memory, so results
// never depend on the prediction.
#pragma once

#include "mulo_dense.cuh"

namespace mulo {

// ------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// global -> shared bulk copy (16-byte aligned, size a multiple of 16), completion
// counted in bytes on `bar`.  Never multicast.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst_smem)),
               "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

#define MULO_DEV_TIMEOUT_BIT MULO_DEV_TIMEOUT
constexpr uint32_t kSpinLimit = 1u << 24;   // bounded waits: give up, flag, carry on

__device__ __forceinline__ void mbar_wait(uint64_t* bar, uint32_t parity, uint32_t* dev_status) {
  for (uint32_t it = 0; it < kSpinLimit; ++it)
    if (mbar_try_wait(bar, parity)) return;
  atomicOr(dev_status, MULO_DEV_TIMEOUT_BIT);   // the data is then garbage, but nothing hangs
}

// ------------------------------------------------------------ configuration
constexpr int kPiece = 256;          // elements per warp visit: 32 lanes x 8
constexpr int kStages = 3;           // ring slots
constexpr int kBins = 512;           // selection histogram bins (= kThreads)
constexpr int kMemberCap = 128;      // entries of the crossing bin ranked exactly

struct SparseArgs {
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
  int n_parents;
  int chunk;        // elements per ring slot (multiple of kPiece)
  int n_chunks;     // chunks per row = ceil(V / chunk)
  int cap;          // candidate capacity (multiple of 16)
  int n_seg;        // segments per row = n_chunks * (chunk / kPiece)
  int margin;       // extra candidates aimed for in steady state
  int margin_boot;  // extra candidates aimed for when no prediction exists
  float a_theta;    // Phi^-1(1 - k/V)
  float a_boot;     // Phi^-1(1 - (k + margin_boot)/V)
  float phi_theta;  // standard normal density at a_theta
};

// Pivot predictor of one kind of row (draft rows / target rows), per CTA:
// the running k-th largest value and the density of entries just below it.
struct Predictor {
  int have;
  float theta, rho;
};

struct SparseSmem {
  // control
  uint64_t full[kStages];
  uint64_t empty[kStages];
  unsigned hist[kBins];
  float members[kMemberCap];
  unsigned n_cand;        // candidates written by the streaming pass
  unsigned n_member;
  unsigned overflow;
  int tok_idx;            // index of x~ in the candidate list, or -1
  uint32_t rnd[4];
};

// Carved from dynamic shared memory (all sizes known on the host).
struct SparseViews {
  unsigned char* ring;    // kStages slots of slot_bytes
  float* tz;              // [cap]  target candidates: z, later e = exp(z - m)
  uint16_t* tid;          // [cap]  their token ids
  float* qz;              // [cap]  draft candidates: z, later qe
  uint16_t* t_start;      // [n_seg] first entry of a segment (target row)
  uint16_t* t_cnt;        // [n_seg]
  uint16_t* q_start;      // [n_seg]
  uint16_t* q_cnt;        // [n_seg]
  uint8_t* q_bits;        // [V/8]   8-entry survivor masks of the draft row
  uint8_t* q_off;         // [V/8]   entries of the segment before each mask
  double* seg_a;          // [n_seg] per-segment sums of e
  double* seg_b;          // [n_seg] per-segment sums of residual weights
};

__host__ __device__ inline size_t sparse_align(size_t x) { return (x + 127) / 128 * 128; }

__host__ __device__ inline size_t sparse_layout(const SparseArgs& a, size_t slot_bytes, SparseViews* v,
                                                unsigned char* base) {
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off += sparse_align(bytes);
    return o;
  };
  size_t o_ring = take(slot_bytes * kStages);
  size_t o_tz = take((size_t)a.cap * 4), o_tid = take((size_t)a.cap * 2), o_qz = take((size_t)a.cap * 4);
  size_t o_ts = take((size_t)a.n_seg * 2), o_tc = take((size_t)a.n_seg * 2);
  size_t o_qs = take((size_t)a.n_seg * 2), o_qc = take((size_t)a.n_seg * 2);
  size_t o_qb = take((size_t)a.n_seg * 32), o_qo = take((size_t)a.n_seg * 32);
  size_t o_sa = take((size_t)a.n_seg * 8), o_sb = take((size_t)a.n_seg * 8);
  if (v) {
    v->ring = base + o_ring;
    v->tz = (float*)(base + o_tz);
    v->tid = (uint16_t*)(base + o_tid);
    v->qz = (float*)(base + o_qz);
    v->t_start = (uint16_t*)(base + o_ts);
    v->t_cnt = (uint16_t*)(base + o_tc);
    v->q_start = (uint16_t*)(base + o_qs);
    v->q_cnt = (uint16_t*)(base + o_qc);
    v->q_bits = (uint8_t*)(base + o_qb);
    v->q_off = (uint8_t*)(base + o_qo);
    v->seg_a = (double*)(base + o_sa);
    v->seg_b = (double*)(base + o_sb);
  }
  return off;
}

// eight pre-processed logits of one lane from a ring slot
template <bool BF16, bool HAS_U>
__device__ __forceinline__ void slot_load8(const unsigned char* slot, int chunk_elems, int e, float s,
                                           float invT, float (&z)[8]) {
  if (BF16) {
    uint4 c = *reinterpret_cast<const uint4*>(slot + (size_t)e * 2);
    uint4 u = make_uint4(0, 0, 0, 0);
    if (HAS_U) u = *reinterpret_cast<const uint4*>(slot + (size_t)chunk_elems * 2 + (size_t)e * 2);
    z[0] = mix_logit(bf16_lo(c.x), bf16_lo(u.x), HAS_U, s, invT);
    z[1] = mix_logit(bf16_hi(c.x), bf16_hi(u.x), HAS_U, s, invT);
    z[2] = mix_logit(bf16_lo(c.y), bf16_lo(u.y), HAS_U, s, invT);
    z[3] = mix_logit(bf16_hi(c.y), bf16_hi(u.y), HAS_U, s, invT);
    z[4] = mix_logit(bf16_lo(c.z), bf16_lo(u.z), HAS_U, s, invT);
    z[5] = mix_logit(bf16_hi(c.z), bf16_hi(u.z), HAS_U, s, invT);
    z[6] = mix_logit(bf16_lo(c.w), bf16_lo(u.w), HAS_U, s, invT);
    z[7] = mix_logit(bf16_hi(c.w), bf16_hi(u.w), HAS_U, s, invT);
  } else {
    const float4* cp = reinterpret_cast<const float4*>(slot + (size_t)e * 4);
    float4 c0 = cp[0], c1 = cp[1];
    float4 u0 = make_float4(0, 0, 0, 0), u1 = u0;
    if (HAS_U) {
      const float4* up = reinterpret_cast<const float4*>(slot + (size_t)chunk_elems * 4 + (size_t)e * 4);
      u0 = up[0];
      u1 = up[1];
    }
    z[0] = mix_logit(c0.x, u0.x, HAS_U, s, invT);
    z[1] = mix_logit(c0.y, u0.y, HAS_U, s, invT);
    z[2] = mix_logit(c0.z, u0.z, HAS_U, s, invT);
    z[3] = mix_logit(c0.w, u0.w, HAS_U, s, invT);
    z[4] = mix_logit(c1.x, u1.x, HAS_U, s, invT);
    z[5] = mix_logit(c1.y, u1.y, HAS_U, s, invT);
    z[6] = mix_logit(c1.z, u1.z, HAS_U, s, invT);
    z[7] = mix_logit(c1.w, u1.w, HAS_U, s, invT);
  }
}

__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}

// Sum of a per-segment double array in a fixed order; every lane of the calling
// warp gets the same value.
__device__ __forceinline__ double warp_total(const double* seg, int n_seg) {
  double t = 0.0;
  for (int s = threadIdx.x & 31; s < n_seg; s += 32) t += seg[s];
  return warp_sum(t);
}

// draft-row lookup: value stored for token id (qe after the draft row's post
// pass), or 0 when the id is not among the draft candidates
__device__ __forceinline__ float q_lookup(const SparseViews& v, int id) {
  const int seg = id >> 8, cell = id >> 3, j = id & 7;
  const unsigned m = v.q_bits[cell];
  if (!((m >> j) & 1u)) return 0.0f;
  const int rank = v.q_off[cell] + __popc(m & ((1u << j) - 1u));
  return v.qz[v.q_start[seg] + rank];
}

// Exact k-th largest among the candidates, given the histogram the streaming
// pass filled over [pivot, pivot + kBins / inv_w).  Every warp runs the same
// scan, so no broadcast is needed.  Returns false (block-uniform) if the rank
// falls outside the histogram or the crossing bin is too crowded.
//   theta: the k-th largest value; n_ge: number of candidates >= theta.
struct SelectResult {
  bool ok;
  float theta;
  int n_ge;
};

__device__ inline SelectResult select_kth(const float* cz, int n, int k, float pivot, float inv_w,
                                          SparseSmem& sm) {
  SelectResult r;
  r.ok = false;
  r.theta = 0.f;
  r.n_ge = 0;
  const int lane = threadIdx.x & 31;
  const int rank = n - k + 1;   // 1-based rank from the bottom of the k-th largest
  // bins [lane*16, lane*16+16)
  unsigned mine = 0;
#pragma unroll
  for (int b = 0; b < kBins / 32; ++b) mine += sm.hist[lane * (kBins / 32) + b];
  unsigned inc = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    unsigned t = __shfl_up_sync(kFull, inc, o);
    if (lane >= o) inc += t;
  }
  const unsigned total_in = __shfl_sync(kFull, inc, 31);
  if ((unsigned)rank > total_in) return r;   // beyond the histogram range
  const unsigned owner_mask = __ballot_sync(kFull, inc >= (unsigned)rank);
  const int owner = __ffs(owner_mask) - 1;
  unsigned before = inc - mine;   // entries in bins of lower lanes
  int bstar = 0;
  unsigned cum = 0;
  if (lane == owner) {
    cum = before;
    for (int b = 0; b < kBins / 32; ++b) {
      unsigned hcnt = sm.hist[lane * (kBins / 32) + b];
      if (cum + hcnt >= (unsigned)rank) {
        bstar = lane * (kBins / 32) + b;
        break;
      }
      cum += hcnt;
    }
  }
  bstar = __shfl_sync(kFull, bstar, owner);
  cum = __shfl_sync(kFull, cum, owner);
  const unsigned in_bin = sm.hist[bstar];
  if (in_bin > (unsigned)kMemberCap) return r;
  // collect the members of the crossing bin (block-wide), then rank them
  for (int i = threadIdx.x; i < n; i += kThreads) {
    float z = cz[i];
    float fb = (z - pivot) * inv_w;
    if (fb < (float)kBins && (int)fb == bstar) {
      unsigned slot = atomicAdd(&sm.n_member, 1u);
      if (slot < (unsigned)kMemberCap) sm.members[slot] = z;
    }
  }
  __syncthreads();
  const int mcount = (int)min(sm.n_member, (unsigned)kMemberCap);
  const int want = rank - (int)cum;   // 1-based rank inside the bin
  float theta = 0.f;
  int less_at = 0;
  bool hit = false;
  for (int i = lane; i < mcount; i += 32) {
    float vi = sm.members[i];
    int less = 0, leq = 0;
    for (int j = 0; j < mcount; ++j) {
      float vj = sm.members[j];
      less += vj < vi;
      leq += vj <= vi;
    }
    if (less < want && want <= leq) {
      theta = vi;
      less_at = less;
      hit = true;
    }
  }
  const unsigned hm = __ballot_sync(kFull, hit);
  if (hm == 0 || mcount != (int)in_bin) return r;
  const int src = __ffs(hm) - 1;
  r.theta = __shfl_sync(kFull, theta, src);
  r.n_ge = n - (int)cum - __shfl_sync(kFull, less_at, src);
  r.ok = true;
  return r;
}

// First index within [0, cnt) of a segment whose running weight sum exceeds y
// (one warp; weights from `wfun(i)`), or the last index with weight if rounding
// leaves the sum short.  Returns -1 for an empty / weightless segment.
template <class W>
__device__ __forceinline__ int warp_locate(int cnt, float y, W wfun) {
  const int lane = threadIdx.x & 31;
  float carry = 0.f;
  int last_pos = -1;
  for (int base = 0; base < cnt; base += 32) {
    const int i = base + lane;
    float w = i < cnt ? wfun(i) : 0.f;
    float inc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      float t = __shfl_up_sync(kFull, inc, o);
      if (lane >= o) inc += t;
    }
    const unsigned hit = __ballot_sync(kFull, w > 0.f && carry + inc > y);
    if (hit) return base + __ffs(hit) - 1;
    const unsigned pos = __ballot_sync(kFull, w > 0.f);
    if (pos) last_pos = base + 31 - __clz(pos);
    carry += __shfl_sync(kFull, inc, 31);
  }
  return last_pos;
}

// One inverse-CDF draw over per-segment weight sums `seg` (ascending id):
// warp 0 scans the segment sums in double, finds the segment that holds
// u * total, then the entry inside it.  Returns the candidate index, or -1
// when the total is zero.  Call from all lanes of ONE warp.
template <class W>
__device__ inline int warp_draw(const double* seg, int n_seg, const uint16_t* start, const uint16_t* cnt,
                                double u, W wfun) {
  const int lane = threadIdx.x & 31;
  // exclusive scan over segments, 32 at a time
  double total = 0.0;
  for (int s = lane; s < n_seg; s += 32) total += seg[s];
  total = warp_sum(total);
  if (!(total > 0.0)) return -1;
  const double y = u * total;
  double carry = 0.0;
  int last_seg = -1;
  for (int base = 0; base < n_seg; base += 32) {
    const int s = base + lane;
    double w = s < n_seg ? seg[s] : 0.0;
    double inc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      double t = __shfl_up_sync(kFull, inc, o);
      if (lane >= o) inc += t;
    }
    const unsigned hit = __ballot_sync(kFull, w > 0.0 && carry + inc > y);
    if (hit) {
      const int l = __ffs(hit) - 1;
      const int sseg = base + l;
      const double before = carry + __shfl_sync(kFull, inc - w, l);
      const int at = warp_locate((int)cnt[sseg], (float)(y - before), [&](int i) { return wfun((int)start[sseg] + i); });
      if (at >= 0) return (int)start[sseg] + at;
    }
    const unsigned pos = __ballot_sync(kFull, w > 0.0);
    if (pos) last_seg = base + 31 - __clz(pos);
    carry += __shfl_sync(kFull, inc, 31);
  }
  if (last_seg < 0) return -1;
  // rounding left u * total at (or past) the end: the last entry with weight
  const int at = warp_locate((int)cnt[last_seg], 3.0e38f, [&](int i) { return wfun((int)start[last_seg] + i); });
  return at >= 0 ? (int)start[last_seg] + at : -1;
}

template <bool BF16, bool HAS_U>
__global__ void __launch_bounds__(kThreads, 2) k_round_sparse(SparseArgs a) {
  __shared__ BlockScratch bs;   // used by the dense fallback
  __shared__ SparseSmem sm;
  extern __shared__ __align__(128) unsigned char dyn[];
  const DevParams& P = a.P;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int esz = BF16 ? 2 : 4;
  const int V = P.V, k = P.top_k, N = P.H * P.W;
  const int rr = P.r * P.r, rows_per_parent = 1 + rr;
  const int pieces = a.chunk / kPiece;
  const size_t slot_bytes = (size_t)a.chunk * esz * 2;   // cond + uncond halves
  SparseViews v;
  sparse_layout(a, slot_bytes, &v, dyn);

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.full[s], 1);
      mbar_init(&sm.empty[s], kWarps);
    }
    mbar_fence_init();
    sm.n_cand = 0;
    sm.n_member = 0;
    sm.overflow = 0;
    sm.tok_idx = -1;
  }
  sm.hist[tid] = 0;   // kBins == kThreads
  __syncthreads();

  const int my_parents = ((int)blockIdx.x < a.n_parents) ? (a.n_parents - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  const long long total_chunks = (long long)my_parents * rows_per_parent * a.n_chunks;

  // ---- producer (thread 0): chunk sequence number -> global addresses
  long long issued = 0;
  auto issue_until = [&](long long limit) {
    while (issued < limit && issued < total_chunks) {
      const int slot = (int)(issued % kStages);
      const long long use = issued / kStages;
      if (use > 0) mbar_wait(&sm.empty[slot], (uint32_t)((use - 1) & 1), a.dev_status);
      const long long row_seq = issued / a.n_chunks;
      const int c = (int)(issued % a.n_chunks);
      const int iter = (int)(row_seq / rows_per_parent), j = (int)(row_seq % rows_per_parent);
      const int parent = (int)blockIdx.x + iter * (int)gridDim.x;
      const int elems = min(a.chunk, V - c * a.chunk);
      const uint32_t bytes = (uint32_t)elems * esz;
      unsigned char* dst = v.ring + (size_t)slot * slot_bytes;
      if (j == 0) {
        mbar_expect_tx(&sm.full[slot], bytes);
        bulk_load(dst, a.draft + ((size_t)parent * V + (size_t)c * a.chunk) * esz, bytes, &sm.full[slot]);
      } else {
        const int b = parent / (P.h * P.w), rem = parent % (P.h * P.w), ca = rem / P.w, cc = rem % P.w;
        const int di = (j - 1) / P.r, dj = (j - 1) % P.r;
        const size_t g = (size_t)b * N + (size_t)(ca * P.r + di) * P.W + (size_t)cc * P.r + dj;
        const size_t off = (g * V + (size_t)c * a.chunk) * esz;
        mbar_expect_tx(&sm.full[slot], HAS_U ? 2 * bytes : bytes);
        bulk_load(dst, a.cond + off, bytes, &sm.full[slot]);
        if (HAS_U) bulk_load(dst + (size_t)a.chunk * esz, a.uncond + off, bytes, &sm.full[slot]);
      }
      ++issued;
    }
  };
  if (tid == 0) issue_until(kStages);

  Predictor pred_q = {0, 0.f, 1.f}, pred_t = {0, 0.f, 1.f};
  long long seq = 0;   // next chunk this CTA consumes

  // Streams one row through the ring.  Candidates (z >= pivot) go to (cz, cid)
  // in segments (one per 256-element piece, ascending id inside), survivors are
  // also counted into the selection histogram.  With `boot` the pivot is first
  // estimated from the mean and spread of the row's first chunk.
  auto stream_row = [&](bool is_q, Predictor& pr, float* cz, uint16_t* cid, uint16_t* sstart, uint16_t* scnt,
                        float& pivot, float& inv_w) {
    const float s_cfg = P.cfg_scale, invT = P.invT;
    const bool has_u_row = HAS_U && !is_q;
    if (pr.have) {
      const float d = (float)a.margin / pr.rho;
      pivot = pr.theta - d;
      inv_w = (float)kBins / (4.0f * d);
    } else {
      // wait for the first chunk (without releasing it) and take its mean / spread
      if (tid == 0) issue_until(seq + kStages);
      mbar_wait(&sm.full[seq % kStages], (uint32_t)((seq / kStages) & 1), a.dev_status);
      const unsigned char* slot = v.ring + (size_t)(seq % kStages) * slot_bytes;
      const int elems = min(a.chunk, V);
      float s1 = 0.f, s2 = 0.f;
      for (int e = tid * 8; e < elems; e += kThreads * 8) {
        float z[8];
        if (has_u_row) slot_load8<BF16, true>(slot, a.chunk, e, s_cfg, invT, z);
        else slot_load8<BF16, false>(slot, a.chunk, e, s_cfg, invT, z);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          s1 += z[j];
          s2 += z[j] * z[j];
        }
      }
      const double S1 = block_sum((double)s1, bs), S2 = block_sum((double)s2, bs);
      const float mean = (float)(S1 / elems);
      const float sd = sqrtf(fmaxf((float)(S2 / elems) - mean * mean, 1e-20f));
      pivot = mean + a.a_boot * sd;
      const float span = 2.5f * (a.a_theta - a.a_boot) * sd;
      inv_w = (float)kBins / fmaxf(span, 1e-20f);
    }
    for (int c = 0; c < a.n_chunks; ++c, ++seq) {
      if (tid == 0) issue_until(seq + kStages);
      const int slot_i = (int)(seq % kStages);
      mbar_wait(&sm.full[slot_i], (uint32_t)((seq / kStages) & 1), a.dev_status);
      const unsigned char* slot = v.ring + (size_t)slot_i * slot_bytes;
      for (int piece = warp; piece < pieces; piece += kWarps) {
        const int seg = c * pieces + piece;
        const int e = piece * kPiece + lane * 8;
        const int id0 = c * a.chunk + e;
        float z[8];
        unsigned mask = 0;
        if (id0 < V) {
          if (has_u_row) slot_load8<BF16, true>(slot, a.chunk, e, s_cfg, invT, z);
          else slot_load8<BF16, false>(slot, a.chunk, e, s_cfg, invT, z);
#pragma unroll
          for (int j = 0; j < 8; ++j) mask |= (z[j] >= pivot ? 1u : 0u) << j;
        }
        const int cnt = __popc(mask);
        int inc = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          int t = __shfl_up_sync(kFull, inc, o);
          if (lane >= o) inc += t;
        }
        const int total = __shfl_sync(kFull, inc, 31);
        int base = 0;
        if (lane == 0) {
          base = (int)atomicAdd(&sm.n_cand, (unsigned)total);
          sstart[seg] = (uint16_t)min(base, 65535);
          scnt[seg] = (uint16_t)total;
          if (base + total > a.cap) sm.overflow = 1;
        }
        base = __shfl_sync(kFull, base, 0);
        const int off = inc - cnt;
        if (is_q && id0 < V) {
          v.q_bits[id0 >> 3] = (uint8_t)mask;
          v.q_off[id0 >> 3] = (uint8_t)min(off, 255);
        }
        int pos = base + off;
        if (base + total <= a.cap) {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if ((mask >> j) & 1u) {
              cz[pos] = z[j];
              if (cid) cid[pos] = (uint16_t)(id0 + j);
              const float fb = (z[j] - pivot) * inv_w;
              if (fb < (float)kBins) atomicAdd(&sm.hist[(int)fb], 1u);
              ++pos;
            }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.empty[slot_i]);
    }
  };

  // Updates the predictor after a row (ok: exact theta found among n candidates).
  auto learn = [&](Predictor& pr, bool ok, float theta, float pivot, int n, int n_ge) {
    if (!ok) {
      pr.have = 0;
      return;
    }
    const int below = n - n_ge;   // candidates in [pivot, theta)
    float rho = pr.rho;
    bool rho_ok = pr.have != 0;
    if (theta > pivot && below >= 16) {
      const float r_new = (float)below / (theta - pivot);
      rho = pr.have ? pr.rho + 0.25f * (r_new - pr.rho) : r_new;
      rho_ok = true;
    }
    if (!rho_ok) {   // no usable density yet: stay in bootstrap mode
      pr.have = 0;
      return;
    }
    pr.theta = pr.have ? pr.theta + 0.25f * (theta - pr.theta) : theta;
    pr.rho = rho;
    pr.have = 1;
  };

  for (int iter = 0; iter < my_parents; ++iter) {
    const int parent = (int)blockIdx.x + iter * (int)gridDim.x;
    const int b = parent / (P.h * P.w), rem = parent % (P.h * P.w), ca = rem / P.w, cc = rem % P.w;
    const int tok = checked_token(a.draft_tok_lo[parent], V, a.dev_status);
    RowSrc qr;
    qr.cond = a.draft + (size_t)parent * V * esz;
    qr.uncond = nullptr;
    qr.s = 0.f;
    qr.invT = P.invT;
    qr.V = V;
    qr.bf16 = BF16;

    // ------------------------------------------------------------ draft row
    RowStats sq;
    bool q_sparse;
    float qe_tok = 0.f;   // exp(z_q(x~) - m_q) or 0
    {
      float pivot, inv_w;
      stream_row(true, pred_q, v.qz, nullptr, v.q_start, v.q_cnt, pivot, inv_w);
      __syncthreads();
      if (tid == 0) issue_until(seq + kStages);   // every slot is free now: prefetch the next row
      const int n = (int)sm.n_cand;
      bool ok = !sm.overflow && n >= k;
      SelectResult sel;
      sel.ok = false;
      if (ok) sel = select_kth(v.qz, n, k, pivot, inv_w, sm);   // contains a barrier when it gets that far
      ok = ok && sel.ok;
      // block-uniform: every warp ran the same scan on the same data
      __syncthreads();
      if (ok) {
        // m_q, then qe = exp(z - m_q) for survivors (0 for the band below theta_q), Z_q
        float mx = -INFINITY;
        for (int i = tid; i < n; i += kThreads) mx = fmaxf(mx, v.qz[i]);
        sq.m = block_max(mx, bs);
        sq.theta = sel.theta;
        for (int s = warp; s < a.n_seg; s += kWarps) {
          const int st = v.q_start[s], cn = v.q_cnt[s];
          float acc = 0.f;
          for (int i = lane; i < cn; i += 32) {
            const float z = v.qz[st + i];
            const float e = z >= sel.theta ? expf(__fsub_rn(z, sq.m)) : 0.f;
            v.qz[st + i] = e;
            acc += e;
          }
          const double tot = warp_sum((double)acc);
          if (lane == 0) v.seg_a[s] = tot;
        }
        __syncthreads();
        sq.Z = warp_total(v.seg_a, a.n_seg);
        qe_tok = q_lookup(v, tok);
      }
      learn(pred_q, ok, sel.theta, pivot, n, sel.n_ge);
      q_sparse = ok;
      __syncthreads();
      if (tid == 0) {
        sm.n_cand = 0;
        sm.n_member = 0;
        sm.overflow = 0;
      }
      sm.hist[tid] = 0;
      if (!ok) {
        if (tid == 0) atomicOr(a.dev_status, MULO_DEV_DENSE_FALLBACK);
        dense_row_stats(qr, k, bs, sq.theta, sq.m, sq.Z);
      }
      {   // same rounding of Z_q as the unfused path (fp32 hi + lo)
        const float Zhi = (float)sq.Z, Zlo = (float)(sq.Z - (double)Zhi);
        sq.Z = (double)Zhi + (double)Zlo;
      }
      __syncthreads();
    }
    const double q_tok = q_sparse ? (double)qe_tok / sq.Z
                                  : ((load1(qr, tok) >= sq.theta) ? exp((double)load1(qr, tok) - (double)sq.m) / sq.Z : 0.0);
    if (q_tok <= 0.0 && tid == 0) atomicOr(a.dev_status, MULO_DEV_ZERO_DRAFT_PROB);
    const float invZq = (float)(1.0 / sq.Z);

    // ------------------------------------------------------------ children
    for (int child = 0; child < rr; ++child) {
      const int t = (ca * P.r + child / P.r) * P.W + cc * P.r + child % P.r;
      const size_t g = (size_t)b * N + t;
      const uint32_t image = (uint32_t)b + P.image_offset;
      if (tid == 32) {   // uniforms of this position, ready long before they are needed
        uint4 r = philox4x32_10(make_uint4((uint32_t)t, image, P.round, 0u), make_uint2(P.seed_lo, P.seed_hi));
        sm.rnd[0] = r.x;
        sm.rnd[1] = r.y;
        sm.rnd[2] = r.z;
        sm.tok_idx = -1;
      }
      float pivot, inv_w;
      stream_row(false, pred_t, v.tz, v.tid, v.t_start, v.t_cnt, pivot, inv_w);
      __syncthreads();
      if (tid == 0) issue_until(seq + kStages);
      const int n = (int)sm.n_cand;
      bool ok = q_sparse && !sm.overflow && n >= k;
      SelectResult sel;
      sel.ok = false;
      if (ok) sel = select_kth(v.tz, n, k, pivot, inv_w, sm);
      ok = ok && sel.ok;
      __syncthreads();
      learn(pred_t, sel.ok, sel.theta, pivot, n, sel.n_ge);
      if (tid == 0) {
        sm.n_cand = 0;
        sm.n_member = 0;
        sm.overflow = 0;
      }
      sm.hist[tid] = 0;

      PositionOut o;
      if (ok) {
        // ---- m_p, e = exp(z - m_p) for survivors, per-segment sums, x~'s entry
        float mx = -INFINITY;
        for (int i = tid; i < n; i += kThreads) mx = fmaxf(mx, v.tz[i]);
        const float m_p = block_max(mx, bs);
        for (int s = warp; s < a.n_seg; s += kWarps) {
          const int st = v.t_start[s], cn = v.t_cnt[s];
          float acc = 0.f;
          for (int i = lane; i < cn; i += 32) {
            const float z = v.tz[st + i];
            const float e = z >= sel.theta ? expf(__fsub_rn(z, m_p)) : 0.f;
            v.tz[st + i] = e;
            acc += e;
            if ((int)v.tid[st + i] == tok) sm.tok_idx = st + i;
          }
          const double tot = warp_sum((double)acc);
          if (lane == 0) v.seg_a[s] = tot;
        }
        __syncthreads();
        // ---- decision, computed identically by every warp
        const double Zp = warp_total(v.seg_a, a.n_seg);
        const float invZp = (float)(1.0 / Zp);
        const int ti = sm.tok_idx;
        const double p_tok = ti >= 0 ? (double)v.tz[ti] / Zp : 0.0;
        double thr;
        int accepted;
        if (P.accept_mode == MULO_ACCEPT_THRESHOLD) {
          thr = p_tok;
          accepted = p_tok >= P.tau;
        } else {
          if (q_tok <= 0.0) thr = p_tok > 0.0 ? 1.0 : 0.0;
          else thr = fmin(1.0, p_tok / q_tok);
          accepted = uniform24(sm.rnd[0]) < thr;
        }
        const int draws = draws_for(P.resample_mode, accepted);
        auto w_target = [&](int i) { return __fmul_rn(v.tz[i], invZp); };
        auto w_resid = [&](int i) {
          const float pe = __fmul_rn(v.tz[i], invZp);
          const float qv = __fmul_rn(q_lookup(v, (int)v.tid[i]), invZq);
          return fmaxf(__fsub_rn(pe, qv), 0.f);
        };
        if (draws & kDrawResidual) {
          for (int s = warp; s < a.n_seg; s += kWarps) {
            const int st = v.t_start[s], cn = v.t_cnt[s];
            float acc = 0.f;
            for (int i = lane; i < cn; i += 32) acc += w_resid(st + i);
            const double tot = warp_sum((double)acc);
            if (lane == 0) v.seg_b[s] = tot;
          }
        }
        __syncthreads();
        int t_res = -1, t_tgt = -1;
        if (warp == 0) {
          if (draws & kDrawResidual) {
            int at = warp_draw(v.seg_b, a.n_seg, v.t_start, v.t_cnt, uniform24(sm.rnd[1]), w_resid);
            if (at < 0)   // residual without mass: the target weights, same uniform
              at = warp_draw(v.seg_a, a.n_seg, v.t_start, v.t_cnt, uniform24(sm.rnd[1]),
                             [&](int i) { return v.tz[i]; });
            t_res = at >= 0 ? (int)v.tid[at] : -1;
          }
        } else if (warp == 1) {
          if (draws & kDrawTarget) {
            const int at = warp_draw(v.seg_a, a.n_seg, v.t_start, v.t_cnt, uniform24(sm.rnd[2]),
                                     [&](int i) { return v.tz[i]; });
            t_tgt = at >= 0 ? (int)v.tid[at] : -1;
          }
        }
        if (warp == 0 && lane == 0) {
          a.flags[g] = accepted ? 0 : 1;
          a.cand_res[g] = t_res;
          if (a.p_tok) a.p_tok[g] = (float)p_tok;
          if (a.q_tok) a.q_tok[g] = (float)q_tok;
          if (a.accept_prob) a.accept_prob[g] = (float)thr;
        }
        if (warp == 1 && lane == 0) a.cand_tgt[g] = t_tgt;
        __syncthreads();
      } else {
        __syncthreads();
        if (tid == 0) atomicOr(a.dev_status, MULO_DEV_DENSE_FALLBACK);
        RowSrc tr;
        const size_t rb = (size_t)V * esz;
        tr.cond = a.cond + g * rb;
        tr.uncond = HAS_U ? a.uncond + g * rb : nullptr;
        tr.s = P.cfg_scale;
        tr.invT = P.invT;
        tr.V = V;
        tr.bf16 = BF16;
        const int mode = P.resample_mode;
        PoolSmem none = {nullptr, nullptr};
        dense_position(P, tr, qr, sq, tok, nullptr, image, (uint32_t)t, true, 0,
                       [mode](int acc) { return draws_for(mode, acc); }, bs, none, a.dev_status, o);
        if (tid == 0) {
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
  }
}

}  // namespace mulo
