// The fast path of the fused round for rows with top-k on (no pooling).
//
// A persistent CTA (256 threads, three per SM) owns a contiguous range of parent
// (low-res) cells.  For each parent it streams the draft row and then its r*r
// target rows ONCE through a shared-memory ring filled by bulk-async copies
// (cp.async.bulk + mbarrier); the warp that releases a slot last requests the next
// chunk into it, so there is no producer thread to wait for.  A chunk iteration has
// a fixed latency of several hundred cycles (barrier wait, shared loads, release),
// so every warp works on two independent 32-lane pieces of the row per iteration
// and releases the slot as soon as its data are in registers; the kernel is bound
// by instruction issue and latency, which is why it is shaped for three resident
// CTAs per SM (80 registers per thread, under 78 KB of shared memory).
// The streaming pass keeps only the entries above a predicted pivot (k plus a
// margin) and appends them, in ascending token id, to the list of their piece of
// the row ("segment"); a segment's list is a run of one array shared by the row,
// claimed with one atomic add.  Everything else -- the exact k-th largest value,
// softmax, acceptance, residual and the inverse-CDF draws -- works on those ~k
// candidates in shared memory.  Each warp post-processes the segments it wrote,
// eight lanes per segment, and values every warp needs (threshold, partition sum,
// accept bit) are recomputed by every warp from shared data instead of being
// broadcast behind a barrier.  A row whose prediction fails (too few candidates, a
// full segment, too many ties at the threshold) is put on a list that a second
// launch works off with the dense routines, so results never depend on the
// prediction and a failed row does not hold up its CTA.
//
// State that is the same for all threads lives in shared memory or in the kernel
// parameters, not in registers.
#pragma once

#include <type_traits>

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

constexpr uint32_t kSpinLimit = 1u << 22;   // bounded waits: give up, flag, carry on

// After a wait has given up, the CTA's abort flag is up: later waits return at once and the
// CTA stops at its next parent (the data is garbage by then, but nothing hangs).
__device__ __forceinline__ void mbar_wait(uint64_t* bar, uint32_t parity, uint32_t* dev_status, volatile int* abort) {
  if (mbar_try_wait(bar, parity)) return;
  if (*abort) return;
#pragma unroll 1
  for (uint32_t it = 0; it < kSpinLimit; ++it)
    if (mbar_try_wait(bar, parity)) return;
  atomicOr(dev_status, MULO_DEV_TIMEOUT);
  *abort = 1;
}

// two fp32 operations per instruction (sm_100 packed fp32); each half is the
// IEEE round-to-nearest result of the scalar operation
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}

// exp(z - m) for the bulk of a row: a subtract, a multiply and one ex2.  Relative
// error about 2^-22 (1 + |z - m|); the probability of the draft token itself,
// which decides acceptance, is computed in double precision.
__device__ __forceinline__ float fast_exp(float z, float m) {
  float r;
  const float t = __fmul_rn(__fsub_rn(z, m), 1.4426950408889634f);
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(t));
  return r;
}

// ------------------------------------------------------------ configuration
constexpr int kSThreads = 256;       // threads per CTA of the streaming kernel
constexpr int kSWarps = kSThreads / 32;
constexpr int kPPW = 2;              // pieces per warp per chunk (independent work per iteration)
constexpr int kChunkPieces = kSWarps * kPPW;
constexpr int kStages = 2;           // ring slots
constexpr int kHistBins = 256;       // selection histogram bins
constexpr int kMemberCap = 128;      // entries of the crossing bin ranked exactly
constexpr int kTableParents = 4;     // parents whose row addresses are kept
constexpr int kMaxRowsPerParent = 17;   // draft row + r*r children, r <= 4
// words of the device status block after the flag word: rows redone by the general
// routines, and why the fast path gave them up
enum : int { kCntRows = 1, kCntListFull = 2, kCntTooFew = 3, kCntAboveRange = 4, kCntCrowdedBin = 5,
             kFailCount = 8 };   // word 8: length of the list of positions left to the dense routines

struct StreamArgs {
  DevParams P;
  const char* cond;
  const char* uncond;
  const char* draft;
  const int32_t* draft_tok_lo;
  const uint16_t* nn;    // pooling: [V, pool_k] neighbour lists (entry 0 of a row is the token itself)
  int32_t* sample_out;   // sampling mode: [B, h, w] the drafter's own draw per low-res cell
  float* p_tok;
  float* q_tok;
  float* accept_prob;
  uint8_t* flags;
  int32_t* cand_res;
  int32_t* cand_tgt;
  uint32_t* dev_status;
  int32_t* fail_list;   // positions b*N + t whose rows the dense routines must do (length at dev_status[kFailCount])
  int n_parents;
  int chunk;        // elements per ring slot half = kChunkPieces pieces
  int n_chunks;     // chunks per row = ceil(V / chunk)
  int n_seg;        // segments per row = n_chunks * kSWarps; segment c * kSWarps + w is the part of chunk c
                    // that warp w handles: kPPW adjacent 32-lane pieces, i.e. kPPW * 32 * (16 / esz) entries
  int cap;          // candidate capacity of a row (all segments together)
  int margin;       // extra candidates aimed for in steady state
  float a_theta;    // Phi^-1(1 - k/V)
  float a_boot;     // Phi^-1(1 - (k + bootstrap margin)/V)
  // byte offsets into dynamic shared memory (computed on the host)
  uint32_t slot_bytes, off_cand, off_qval, off_tseg, off_qseg, off_qcell, off_sega, off_segb, off_segc;
};

inline size_t stream_align(size_t x) { return (x + 127) / 128 * 128; }

// Lays out dynamic shared memory; returns its size.  (host)
inline size_t stream_layout(StreamArgs& a, int esz) {
  const int epl = 16 / esz;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off += stream_align(bytes);
    return (uint32_t)o;
  };
  a.slot_bytes = (uint32_t)((size_t)a.chunk * esz * 2);   // cond + uncond halves
  take((size_t)a.slot_bytes * kStages);                   // the ring sits at offset 0
  a.off_cand = take((size_t)a.cap * 8);   // uint2 (z, later e = exp(z - m); token id) of the target row's candidates
  a.off_qval = take((size_t)a.cap * 4);   // float z, later exp(z - m_q), of the draft row's candidates
  a.off_tseg = take((size_t)a.n_seg * 4); // ushort2 (first entry, entries) per segment, target row
  a.off_qseg = take((size_t)a.n_seg * 4); // the same for the draft row
  a.off_qcell = take((size_t)a.n_chunks * a.chunk / epl * 2);   // uint16 per lane visit of the draft row:
                                                                // survivor mask | (first slot << 8)
  a.off_sega = take((size_t)a.n_seg * 4);   // float per-segment sums of e without the threshold bin's entries
  a.off_segb = take((size_t)a.n_seg * 4);   // float per-segment sums of residual weights
  a.off_segc = take((size_t)a.n_seg * 4);   // float per-segment sums of e, complete
  return off;
}

// Pivot predictor of one kind of row (draft rows / target rows), per CTA:
// the running k-th largest value and the density of entries just below it.
struct Predictor {
  int have;
  float theta, rho;
  float pivot, inv_w;   // what the next row of this kind starts from (valid while have != 0)
  // rows without a prediction take the pivot from the mean and spread of their first chunk,
  // assuming a normal shape; when that start fails, `shift` (in units of the spread) moves the
  // next start down (too few candidates) or up (too many): the step doubles while the
  // failures point the same way and halves when they change direction
  float shift, step;
  int dir;
};

struct RowState {   // selection scratch of the row in work
  unsigned hist[kHistBins];
  float member_z[kMemberCap];
  unsigned short member_at[kMemberCap];
  unsigned short member_seg[kMemberCap];
  unsigned n_cand, n_member, overflow, max_key;
  unsigned alloc;   // entries of the row's candidate array handed out so far
};

struct RowPrep {    // per target row, prepared while the previous row is finished
  uint32_t rnd[3];
  float z_tok;      // pre-processed target logit of x~
};

// Cursor of the next chunk to request into a ring slot: chunk within the row, row within
// the parent, table slot of the parent.  One per ring slot, in shared memory; only the warp
// that is last out of the slot touches it, and two uses of a slot are ordered by the slot's
// own barrier.
struct Cursor {
  int left;          // chunks still to request into this slot
  unsigned pos;      // c | j << 8 | table slot << 16
};
struct StreamSmem {
  uint64_t full[kStages];
  unsigned done[kStages];
  Cursor cursor[kStages];
  RowState rs;
  RowPrep prep[2];
  Predictor pred[2];   // 0: draft rows, 1: target rows
  float red[kSWarps][2];   // bootstrap statistics
  double e_tok;        // exp(z_tok - m_p) of the current target row
  // pooling (Eq. 3-4): warp totals of the prefix scan, first list index whose prefix mass reaches
  // delta, the pooled mass c_J
  double wsum[kSWarps];
  double cJ;
  int first_bad;
  // the current parent
  double Zq, q_tok;
  float theta_q, m_q, invZq;
  int q_ok, tok;
  int b, ca, cc;
  // the parent the address table was last filled for
  int tb, tca, tcc, tparent;
  int abort;           // a wait of this CTA gave up
  unsigned long long row_off[kTableParents][kMaxRowsPerParent];   // byte offsets of the rows within their tensors
};

__device__ __forceinline__ void cursor_advance(Cursor& w, int n_chunks, int rows_per_parent) {
  unsigned c = (w.pos & 0xffu) + 1u, j = (w.pos >> 8) & 0xffu, s = w.pos >> 16;
  if (c == (unsigned)n_chunks) {
    c = 0;
    if (++j == (unsigned)rows_per_parent) {
      j = 0;
      s = (s + 1u) & (kTableParents - 1);
    }
  }
  w.pos = c | (j << 8) | (s << 16);
}

template <bool BF16, bool HAS_U>
__device__ __forceinline__ void cursor_issue(const Cursor& w, const StreamArgs& a, StreamSmem& sm,
                                             unsigned char* ring, int slot) {
  const int esz = BF16 ? 2 : 4;
  const int c = (int)(w.pos & 0xffu), j = (int)((w.pos >> 8) & 0xffu), s = (int)(w.pos >> 16);
  const int elems = min(a.chunk, a.P.V - c * a.chunk);
  const uint32_t bytes = (uint32_t)elems * esz;
  unsigned char* dst = ring + (size_t)slot * a.slot_bytes;
  const size_t off = (size_t)sm.row_off[s][j] + (size_t)c * a.chunk * esz;
  if (j == 0) {
    mbar_expect_tx(&sm.full[slot], bytes);
    bulk_load(dst, a.draft + off, bytes, &sm.full[slot]);
  } else {
    mbar_expect_tx(&sm.full[slot], HAS_U ? 2 * bytes : bytes);
    bulk_load(dst, a.cond + off, bytes, &sm.full[slot]);
    if (HAS_U) bulk_load(dst + (size_t)a.chunk * esz, a.uncond + off, bytes, &sm.full[slot]);
  }
}

// Writes the row offsets of `parent` (coordinates b, ca, cc) into table slot s.
__device__ __forceinline__ void table_fill(const StreamArgs& a, StreamSmem& sm, int s, int parent, int b, int ca,
                                           int cc, int esz) {
  const DevParams& P = a.P;
  const size_t row = (size_t)P.V * esz;
  sm.row_off[s][0] = (unsigned long long)((size_t)parent * row);
  const size_t base = (size_t)b * P.H * P.W + (size_t)ca * P.r * P.W + (size_t)cc * P.r;
  int j = 1;
  for (int di = 0; di < P.r; ++di)
    for (int dj = 0; dj < P.r; ++dj, ++j) sm.row_off[s][j] = (unsigned long long)((base + (size_t)di * P.W + dj) * row);
}

// 16 bytes of the conditional row (8 bf16 or 4 fp32 entries) of one lane, and the same
// entries of the unconditional row, from a ring slot into registers
template <bool BF16, bool HAS_U>
__device__ __forceinline__ void raw_load(const unsigned char* slot, int chunk_elems, int e, uint4& c, uint4& u) {
  constexpr int esz = BF16 ? 2 : 4;
  c = *reinterpret_cast<const uint4*>(slot + (size_t)e * esz);
  u = make_uint4(0, 0, 0, 0);
  if (HAS_U) u = *reinterpret_cast<const uint4*>(slot + (size_t)chunk_elems * esz + (size_t)e * esz);
}
// ... turned into pre-processed logits: d = c - u; v = fma(s, d, u); z = v * invT, each
// one IEEE fp32 rounding (two entries per instruction)
template <bool BF16, bool HAS_U>
__device__ __forceinline__ void raw_mix(const uint4& c, const uint4& u, float s, float invT,
                                        float (&z)[BF16 ? 8 : 4]) {
  const bool scale = invT != 1.0f;
  const uint64_t s2 = pack2(s, s), t2 = pack2(invT, invT);
  if (BF16) {
    const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, uw[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint64_t v = pack2(bf16_lo(cw[i]), bf16_hi(cw[i]));
      if (HAS_U) {
        const uint64_t un = pack2(bf16_lo(uw[i]), bf16_hi(uw[i]));
        v = fma2(s2, sub2(v, un), un);
      }
      if (scale) v = mul2(v, t2);
      unpack2(v, z[2 * i], z[2 * i + 1]);
    }
  } else {
    uint64_t v0 = pack2(__uint_as_float(c.x), __uint_as_float(c.y)), v1 = pack2(__uint_as_float(c.z), __uint_as_float(c.w));
    if (HAS_U) {
      const uint64_t u0 = pack2(__uint_as_float(u.x), __uint_as_float(u.y)), u1 = pack2(__uint_as_float(u.z), __uint_as_float(u.w));
      v0 = fma2(s2, sub2(v0, u0), u0);
      v1 = fma2(s2, sub2(v1, u1), u1);
    }
    if (scale) {
      v0 = mul2(v0, t2);
      v1 = mul2(v1, t2);
    }
    unpack2(v0, z[0], z[1]);
    unpack2(v1, z[2], z[3]);
  }
}

// sum over the `lanes` (a power of two) neighbouring lanes that share a segment
__device__ __forceinline__ float seg_lanes_sum(float v, int lanes) {
  for (int o = 1; o < lanes; o <<= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
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

// One inverse-CDF draw over per-segment weight sums `seg` (segments in ascending
// token id, entries in ascending id inside a segment; `run[s]` = first entry and
// number of entries of segment s): scans the segment sums in double, finds the
// segment that holds u * total, then the entry inside it.  Returns the index into
// the candidate array, or -1 when the total is zero.  Call from all lanes of ONE warp.
template <class W>
__device__ __forceinline__ int warp_draw(const float* seg, int n_seg, const ushort2* run, double u, W wfun,
                                         int* seg_out = nullptr) {
  const int lane = threadIdx.x & 31;
  // every lane sums a block of consecutive segments, then one scan over the lanes
  const int per = (n_seg + 31) / 32;
  const int s0 = lane * per;
  double loc = 0.0;
  for (int i = 0; i < per; ++i)
    if (s0 + i < n_seg) loc += (double)seg[s0 + i];
  double inc = loc;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double t = __shfl_up_sync(kFull, inc, o);
    if (lane >= o) inc += t;
  }
  const double total = __shfl_sync(kFull, inc, 31);
  if (!(total > 0.0)) return -1;
  const double y = u * total;
  const unsigned hit = __ballot_sync(kFull, loc > 0.0 && inc > y);
  // Segments to try, the same in every lane: forward through the block of the lane that holds
  // u * total; then, should rounding have left u * total at (or past) the end, backward from
  // the last segment for the last entry with weight.  One call site for the search inside a
  // segment keeps the code small.
  const int l = hit ? __ffs(hit) - 1 : 0;
  double acc = __shfl_sync(kFull, inc - loc, l);   // mass before lane l's block
  int sidx = hit ? l * per : n_seg - 1;
  const int fwd_end = min((l + 1) * per, n_seg);
  bool forward = hit != 0;
#pragma unroll 1
  for (;;) {
    float yy;
    double w = 0.0;
    if (forward) {
      if (sidx >= fwd_end) {
        forward = false;
        sidx = n_seg - 1;
        continue;
      }
      w = (double)seg[sidx];
      if (!(w > 0.0 && acc + w > y)) {
        acc += w;
        ++sidx;
        continue;
      }
      yy = (float)(y - acc);
    } else {
      if (sidx < 0) return -1;
      if (!(seg[sidx] > 0.f)) {
        --sidx;
        continue;
      }
      yy = 3.0e38f;
    }
    const ushort2 r = run[sidx];
    const int at = warp_locate((int)r.y, yy, [&](int k) { return wfun((int)r.x + k); });
    if (at >= 0) {
      if (seg_out) *seg_out = sidx;
      return (int)r.x + at;
    }
    if (forward) {
      acc += w;
      ++sidx;
    } else {
      --sidx;
    }
  }
}

// where the k-th largest value lies in a row's selection histogram
struct Sel {
  int n;        // candidates streamed
  int bstar;    // the histogram bin that holds the k-th largest
  int want;     // its 1-based rank inside that bin, from below
  int cum;      // entries in the bins below
  float m;      // row maximum
  int reason;   // why the row left the fast path: 0 not at all, 1 list full, 2 too few candidates,
                // 3 k-th largest above the histogram, 4 too many ties at the threshold
};

// SAMPLE = true turns the kernel into the drafter's own sampling (Sec. 3.2 Step 1): only the draft
// rows are streamed (one row per "parent"), and instead of verifying children one warp draws
// y~ ~ q from the row's candidate list with word 0 of the tag-1 Philox stream.
// POOL = true adds the probability pooling of Eq. 3-4 to a target row: the pooled mass of the
// codebook neighbours of x~ enters the acceptance test, and the redraw uses p' (neighbours' mass
// moved onto x~).
template <bool BF16, bool HAS_U, bool SAMPLE = false, bool POOL = false>
__global__ void __launch_bounds__(kSThreads, 3) k_round_stream(const __grid_constant__ StreamArgs a) {
  static_assert(!(SAMPLE && HAS_U), "draft rows have no unconditional stream");
  static_assert(!(SAMPLE && POOL), "the drafter's own draw has no pooling");
  constexpr int EPL = BF16 ? 8 : 4;        // entries per lane visit (16 bytes of the conditional row)
  constexpr int PIECE = 32 * EPL;          // entries per 32-lane piece
  constexpr int SEG = kPPW * PIECE;        // entries of the row that one segment covers
  constexpr int esz = BF16 ? 2 : 4;
  __shared__ StreamSmem sm;
  extern __shared__ __align__(128) unsigned char dyn[];
  const DevParams& P = a.P;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // In the list passes a warp's lanes split into up to four groups, one segment per group
  // at a time (group g takes the warp's segment of chunk g, g + groups, ...).
  const int groups = a.n_chunks >= 3 ? 4 : a.n_chunks;   // 1, 2 or 4
  const int seg_lanes = 32 / groups;
  const int sub = lane & (seg_lanes - 1), grp = lane / seg_lanes;
  unsigned char* const ring = dyn;
  uint2* const cand = reinterpret_cast<uint2*>(dyn + a.off_cand);
  float* const qval = reinterpret_cast<float*>(dyn + a.off_qval);
  ushort2* const tseg = reinterpret_cast<ushort2*>(dyn + a.off_tseg);
  ushort2* const qseg = reinterpret_cast<ushort2*>(dyn + a.off_qseg);
  uint16_t* const qcell = reinterpret_cast<uint16_t*>(dyn + a.off_qcell);
  float* const seg_a = reinterpret_cast<float*>(dyn + a.off_sega);
  float* const seg_b = reinterpret_cast<float*>(dyn + a.off_segb);
  float* const seg_c = reinterpret_cast<float*>(dyn + a.off_segc);
  RowState& rs = sm.rs;

  // this CTA's parents: [p_begin, p_end)
  const int p_begin = (int)(((long long)a.n_parents * blockIdx.x) / gridDim.x);
  const int p_end = (int)(((long long)a.n_parents * (blockIdx.x + 1)) / gridDim.x);
  if (p_end <= p_begin) return;
  const int rr = SAMPLE ? 0 : P.r * P.r, rows_per_parent = 1 + rr;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.full[s], 1);
      sm.done[s] = 0;
    }
    mbar_fence_init();
    sm.abort = 0;
    rs.n_cand = 0;
    rs.n_member = 0;
    rs.overflow = 0;
    rs.max_key = 0;
    rs.alloc = 0;
    for (int s = 0; s < 2; ++s) {
      sm.pred[s].have = 0;
      sm.pred[s].theta = 0.f;
      sm.pred[s].rho = 1.f;
      sm.pred[s].pivot = 0.f;
      sm.pred[s].inv_w = 0.f;
      sm.pred[s].shift = 0.f;
      sm.pred[s].step = 0.f;
      sm.pred[s].dir = 0;
    }
    const int hw = P.h * P.w;
    sm.b = p_begin / hw;
    sm.ca = (p_begin % hw) / P.w;
    sm.cc = (p_begin % hw) % P.w;
    // row addresses of the first three parents
    int tb = sm.b, tca = sm.ca, tcc = sm.cc, tp = p_begin;
    for (int i = 0; i < 3; ++i) {
      if (tp < p_end) table_fill(a, sm, i, tp, tb, tca, tcc, esz);
      if (i == 2) break;
      ++tp;
      if (++tcc == P.w) {
        tcc = 0;
        if (++tca == P.h) {
          tca = 0;
          ++tb;
        }
      }
    }
    sm.tb = tb;
    sm.tca = tca;
    sm.tcc = tcc;
    sm.tparent = tp;
  }
  if (tid < kHistBins) rs.hist[tid] = 0;
  __syncthreads();

  if (tid == 0) {   // the first chunks, and each slot's cursor kStages chunks further on
    const int total = (p_end - p_begin) * rows_per_parent * a.n_chunks;
    Cursor cur;
    cur.pos = 0;
    cur.left = 0;
    for (int s = 0; s < kStages; ++s) {
      if (s < total) cursor_issue<BF16, HAS_U>(cur, a, sm, ring, s);
      Cursor nxt = cur;
      for (int k = 0; k < kStages; ++k) cursor_advance(nxt, a.n_chunks, rows_per_parent);
      nxt.left = total > s + kStages ? (total - s - 1) / kStages : 0;
      sm.cursor[s] = nxt;
      cursor_advance(cur, a.n_chunks, rows_per_parent);
    }
  }
  int rslot = 0;          // ring slot of the next chunk to read
  uint32_t rphase = 0;    // and its phase
  int rowi = 0;           // target rows done so far (selects the RowPrep copy)

  // Releases the slot just read; the last warp out requests the next chunk into it.
  auto release_slot = [&]() {
    __syncwarp();
    if (lane == 0) {
      __threadfence_block();
      const unsigned old = atomicAdd(&sm.done[rslot], 1u);
      if (old == (unsigned)kSWarps - 1u) {
        sm.done[rslot] = 0;
        __threadfence_block();
        Cursor cur = sm.cursor[rslot];
        if (cur.left > 0) {
          cursor_issue<BF16, HAS_U>(cur, a, sm, ring, rslot);
          --cur.left;
#pragma unroll
          for (int k = 0; k < kStages; ++k) cursor_advance(cur, a.n_chunks, rows_per_parent);
          sm.cursor[rslot] = cur;
        }
      }
    }
    if (++rslot == kStages) {
      rslot = 0;
      rphase ^= 1u;
    }
  };

  // Pivot and histogram scale of the next row of a kind.  Without a prediction the
  // pivot is estimated from the mean and spread of the row's first chunk (which
  // stays in its slot for the streaming pass).
  auto choose_pivot = [&](int kind, auto has_u_tag, float& pivot, float& inv_w) {
    constexpr bool ROW_U = decltype(has_u_tag)::value;
    const Predictor pr = sm.pred[kind];
    if (pr.have) {   // block-uniform
      pivot = pr.pivot;
      inv_w = pr.inv_w;
      return;
    }
    mbar_wait(&sm.full[rslot], rphase, a.dev_status, &sm.abort);
    const unsigned char* slot = ring + (size_t)rslot * a.slot_bytes;
    const int elems = min(a.chunk, P.V);
    float s1 = 0.f, s2 = 0.f;
    for (int e = tid * EPL; e < elems; e += kSThreads * EPL) {
      uint4 c, u;
      float z[EPL];
      raw_load<BF16, ROW_U>(slot, a.chunk, e, c, u);
      raw_mix<BF16, ROW_U>(c, u, P.cfg_scale, P.invT, z);
#pragma unroll
      for (int j = 0; j < EPL; ++j) {
        s1 += z[j];
        s2 += z[j] * z[j];
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
    for (int w = 0; w < kSWarps; ++w) {
      S1 += (double)sm.red[w][0];
      S2 += (double)sm.red[w][1];
    }
    __syncthreads();
    const float mean = (float)(S1 / elems);
    const float sd = sqrtf(fmaxf((float)(S2 / elems) - mean * mean, 1e-20f));
    const float d = fmaxf((a.a_theta - a.a_boot) * sd, 1e-20f);
    pivot = mean + (a.a_boot + pr.shift) * sd;
    inv_w = (float)kHistBins / (3.0f * d);
  };

  // Consumes a row's chunks without looking at them (a target row under a draft row
  // that left the fast path).
  auto skip_row = [&]() {
    for (int c = 0; c < a.n_chunks; ++c) {
      mbar_wait(&sm.full[rslot], rphase, a.dev_status, &sm.abort);
      release_slot();
    }
  };

  // Streams one row through the ring: entries with z >= pivot are appended, in ascending
  // token id, to the list of their segment.  Then (pass A) each warp histograms the low end
  // of the lists it wrote and contributes to the row's maximum and candidate count.
  auto stream_row = [&](auto is_q_tag, auto has_u_tag, float pivot, float inv_w) {
    constexpr bool IS_Q = decltype(is_q_tag)::value;
    constexpr bool ROW_U = decltype(has_u_tag)::value;
    ushort2* const run = IS_Q ? qseg : tseg;
    for (int c = 0; c < a.n_chunks; ++c) {
      mbar_wait(&sm.full[rslot], rphase, a.dev_status, &sm.abort);
      const unsigned char* slot = ring + (size_t)rslot * a.slot_bytes;
      uint4 rc[kPPW], ru[kPPW];
#pragma unroll
      for (int i = 0; i < kPPW; ++i) {
        const int e = (kPPW * warp + i) * PIECE + lane * EPL;
        if (c * a.chunk + e < P.V) raw_load<BF16, ROW_U>(slot, a.chunk, e, rc[i], ru[i]);
      }
      release_slot();   // the data are in registers
      unsigned mask[kPPW];
      float z[kPPW][EPL];
#pragma unroll
      for (int i = 0; i < kPPW; ++i) {
        const int e = (kPPW * warp + i) * PIECE + lane * EPL;
        mask[i] = 0;
        if (c * a.chunk + e < P.V) {
          raw_mix<BF16, ROW_U>(rc[i], ru[i], P.cfg_scale, P.invT, z[i]);
#pragma unroll
          for (int j = 0; j < EPL; ++j)
            if (z[i][j] >= pivot) mask[i] |= 1u << j;
          // pooling moves mass onto x~, so x~ gets an entry whatever its value (one that is below
          // the pivot counts for nothing until then: no histogram bin, e = 0)
          if (POOL && !IS_Q) {
            const unsigned d = (unsigned)(sm.tok - (c * a.chunk + e));
            if (d < (unsigned)EPL) mask[i] |= 1u << d;
          }
        }
      }
      // one warp scan for both pieces' counts (16 bits each); lane 31 then claims one run of the
      // row's array for the segment (the two pieces back to back), rounded up to an even length
      // so that runs start on even entries and the list passes can load aligned pairs
      static_assert(kPPW <= 2, "the packed scan below handles at most two pieces");
      const unsigned cnt0 = __popc(mask[0]), cnt1 = kPPW > 1 ? __popc(mask[kPPW - 1]) : 0u;
      unsigned inc = cnt0 | (cnt1 << 16);
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(kFull, inc, o);
        if (lane >= o) inc += t;
      }
      const unsigned tot = __shfl_sync(kFull, inc, 31);
      const int t0 = (int)(tot & 0xffffu), t01 = t0 + (int)(tot >> 16);
      int base = 0;
      if (lane == 31) {
        const int len = (t01 + 1) & ~1;
        base = (int)atomicAdd(&rs.alloc, (unsigned)len);
        // (the draft row's look-up table holds offsets within a segment in 8 bits)
        const bool fits = base + len <= a.cap && (!IS_Q || t01 <= 255);
        run[c * kSWarps + warp] = make_ushort2((unsigned short)(fits ? base : 0), (unsigned short)(fits ? t01 : 0));
        if (!fits) {
          rs.overflow = 1;
          base = -1;
        }
      }
      base = __shfl_sync(kFull, base, 31);
#pragma unroll
      for (int i = 0; i < kPPW; ++i) {
        const int e = (kPPW * warp + i) * PIECE + lane * EPL;
        const int id0 = c * a.chunk + e;
        // position of this lane's first candidate within the segment's run
        const int off = i == 0 ? (int)(inc & 0xffffu) - (int)cnt0 : t0 + (int)(inc >> 16) - (int)cnt1;
        if (IS_Q && id0 < P.V) qcell[id0 / EPL] = (uint16_t)(mask[i] | ((unsigned)min(off, 255) << 8));
        if (base >= 0) {
          if (IS_Q) {
            float* dst = qval + base + off;
#pragma unroll
            for (int j = 0; j < EPL; ++j)
              if ((mask[i] >> j) & 1u) *dst++ = z[i][j];
          } else {
            uint2* dst = cand + base + off;
#pragma unroll
            for (int j = 0; j < EPL; ++j)
              if ((mask[i] >> j) & 1u) *dst++ = make_uint2(__float_as_uint(z[i][j]), (unsigned)(id0 + j));
          }
        }
      }
    }
    // ---- pass A over the lists this warp wrote; a lane takes two pairs of neighbouring entries
    //      per trip, and the group's lanes cover 4 * seg_lanes entries of the segment
    __syncwarp();
    float mx = -INFINITY;
    unsigned mine = 0;
    auto tally = [&](float zz) {
      mx = fmaxf(mx, zz);
      const float fb = __fmul_rn(__fsub_rn(zz, pivot), inv_w);
      if (POOL && !IS_Q) {   // the list may hold x~ from below the pivot: not a candidate
        if (zz >= pivot) {
          ++mine;
          if (fb < (float)kHistBins) atomicAdd(&rs.hist[(int)fb], 1u);
        }
      } else if (fb < (float)kHistBins) {
        atomicAdd(&rs.hist[(int)fb], 1u);
      }
    };
    auto tally_pair = [&](int first, int sl, int cn) {
      float z0, z1;
      if (IS_Q) {
        const float2 v = *reinterpret_cast<const float2*>(qval + first + sl);
        z0 = v.x, z1 = v.y;
      } else {
        const uint4 v = *reinterpret_cast<const uint4*>(cand + first + sl);
        z0 = __uint_as_float(v.x), z1 = __uint_as_float(v.z);
      }
      tally(z0);
      if (sl + 1 < cn) tally(z1);
    };
    for (int c = grp; c < a.n_chunks; c += groups) {
      const ushort2 r = run[c * kSWarps + warp];
      const int cn = r.y;
      if (!(POOL && !IS_Q) && sub == 0) mine += (unsigned)cn;
      for (int sl = 2 * sub; sl < cn; sl += 4 * seg_lanes) {
        tally_pair(r.x, sl, cn);
        if (sl + 2 * seg_lanes < cn) tally_pair(r.x, sl + 2 * seg_lanes, cn);
      }
    }
    __syncwarp();
    const unsigned key = __reduce_max_sync(kFull, float_key(mx));
    mine = __reduce_add_sync(kFull, mine);
    if (lane == 0) {
      atomicMax(&rs.max_key, key);
      if (mine) atomicAdd(&rs.n_cand, mine);
    }
  };

  // After the barrier that follows stream_row: where the k-th largest value lies in
  // the histogram.  Every warp computes the same answer.  false: the row leaves the
  // fast path (block-uniform).
  auto locate_bin = [&](Sel& s) -> bool {
    const int k = P.top_k;
    s.n = (int)rs.n_cand;
    s.reason = 0;
    if (rs.overflow || s.n < k) {
      if (tid == 0) atomicAdd(a.dev_status + (rs.overflow ? kCntListFull : kCntTooFew), 1u);
      s.reason = rs.overflow ? 1 : 2;
      return false;
    }
    s.m = key_float(rs.max_key);
    const int rank = s.n - k + 1;   // 1-based rank from the bottom of the k-th largest
    constexpr int PER = kHistBins / 32;
    unsigned h[PER];
    unsigned mine = 0;
#pragma unroll
    for (int b = 0; b < PER; ++b) {
      h[b] = rs.hist[lane * PER + b];
      mine += h[b];
    }
    unsigned inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned t = __shfl_up_sync(kFull, inc, o);
      if (lane >= o) inc += t;
    }
    const unsigned owner_mask = __ballot_sync(kFull, inc >= (unsigned)rank);
    if (owner_mask == 0) {   // the rank lies above the histogram range
      if (tid == 0) atomicAdd(a.dev_status + kCntAboveRange, 1u);
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
    if (in_bin > (unsigned)kMemberCap) {
      if (tid == 0) atomicAdd(a.dev_status + kCntCrowdedBin, 1u);
      s.reason = 4;
      return false;
    }
    return true;
  };

  // Pass B over the warp's own segments: e = exp(z - m) for every entry at or above the
  // crossing bin (0 below it); the bin's own entries are set aside to be ranked exactly
  // and are left out of the segment sums for now.
  auto exp_pass = [&](auto is_q_tag, const Sel& s, float pivot, float inv_w) {
    constexpr bool IS_Q = decltype(is_q_tag)::value;
    const ushort2* run = IS_Q ? qseg : tseg;
    // e of one entry (value z at index `at`); the crossing bin's entries are set aside
    auto one = [&](int seg, int at, float z, float& acc) -> float {
      const float fb = __fmul_rn(__fsub_rn(z, pivot), inv_w);
      int bin = fb < (float)kHistBins ? (int)fb : kHistBins;
      if (POOL && !IS_Q && z < pivot) bin = -1;   // x~ from below the pivot: e = 0
      float e = 0.f;
      if (bin >= s.bstar) e = fast_exp(z, s.m);
      if (bin == s.bstar) {
        const unsigned slot = atomicAdd(&rs.n_member, 1u);
        if (slot < (unsigned)kMemberCap) {
          rs.member_z[slot] = z;
          rs.member_at[slot] = (unsigned short)at;
          rs.member_seg[slot] = (unsigned short)seg;
        }
      } else {
        acc += e;
      }
      return e;
    };
    // a lane's pair of neighbouring entries of a segment (the second one may lie past its end)
    auto pair = [&](int seg, ushort2 r, int sl, float& acc) {
      const int at = r.x + sl;
      const bool two = sl + 1 < r.y;
      if (IS_Q) {
        float2 v = *reinterpret_cast<float2*>(qval + at);
        v.x = one(seg, at, v.x, acc);
        if (two) v.y = one(seg, at + 1, v.y, acc);
        *reinterpret_cast<float2*>(qval + at) = v;
      } else {
        uint4 v = *reinterpret_cast<uint4*>(cand + at);
        v.x = __float_as_uint(one(seg, at, __uint_as_float(v.x), acc));
        if (two) v.z = __float_as_uint(one(seg, at + 1, __uint_as_float(v.z), acc));
        *reinterpret_cast<uint4*>(cand + at) = v;
      }
    };
    for (int c0 = 0; c0 < a.n_chunks; c0 += groups) {
      const int c = c0 + grp;
      const bool has = c < a.n_chunks;
      const int seg = c * kSWarps + warp;
      float acc = 0.f;
      if (has) {
        const ushort2 r = run[seg];
        for (int sl = 2 * sub; sl < (int)r.y; sl += 4 * seg_lanes) {
          pair(seg, r, sl, acc);
          if (sl + 2 * seg_lanes < (int)r.y) pair(seg, r, sl + 2 * seg_lanes, acc);
        }
      }
      __syncwarp();
      acc = seg_lanes_sum(acc, seg_lanes);
      if (sub == 0 && has) {
        seg_a[seg] = acc;
        if (!IS_Q || SAMPLE) seg_c[seg] = acc;
      }
    }
  };

  // After the barrier that follows exp_pass: the exact k-th largest value theta, the
  // number of entries >= theta, and the partition sum Z (every warp computes the same).
  // Each warp also settles the set-aside entries that lie in its own segments: an entry
  // below theta gets e = 0, one at or above it is added to the complete segment sum.
  auto finish_selection = [&](auto is_q_tag, const Sel& s, float& theta, int& n_ge, double& Z) -> bool {
    constexpr bool IS_Q = decltype(is_q_tag)::value;
    const int mcount = (int)rs.n_member;   // <= kMemberCap: locate_bin checked the bin's size
    float th = 0.f;
    int less_at = 0;
    bool hit = false;
    for (int i = lane; i < mcount; i += 32) {
      const float vi = rs.member_z[i];
      int less = 0, leq = 0;
      for (int jj = 0; jj < mcount; ++jj) {
        const float vj = rs.member_z[jj];
        less += vj < vi;
        leq += vj <= vi;
      }
      if (less < s.want && s.want <= leq) {
        th = vi;
        less_at = less;
        hit = true;
      }
    }
    __syncwarp();
    const unsigned hm = __ballot_sync(kFull, hit);
    if (hm == 0) return false;   // cannot happen: the bin holds the rank
    const int src = __ffs(hm) - 1;
    th = __shfl_sync(kFull, th, src);
    less_at = __shfl_sync(kFull, less_at, src);
    double z = 0.0;
    for (int i = lane; i < mcount; i += 32) {
      const int at = rs.member_at[i], seg = rs.member_seg[i];
      const bool keep = rs.member_z[i] >= th;
      const bool own = (seg & (kSWarps - 1)) == warp;   // one of this warp's segments
      if (keep) {
        const float e = IS_Q ? qval[at] : __uint_as_float(cand[at].x);
        z += (double)e;
        if (own && (!IS_Q || SAMPLE)) {
          // The set-aside slots were handed out in no fixed order.  So that the segment sum does not
          // depend on it, the kept member with the lowest candidate index of a segment adds ALL the
          // segment's kept members at once, summed in double (exact: entries of one histogram bin
          // share their exponent or differ by one).
          bool leader = true;
          double all = 0.0;
          for (int j = 0; j < mcount; ++j)
            if (rs.member_seg[j] == seg && rs.member_z[j] >= th) {
              const int aj = rs.member_at[j];
              leader = leader && aj >= at;
              all += (double)(IS_Q ? qval[aj] : __uint_as_float(cand[aj].x));
            }
          if (leader) seg_c[seg] = (float)((double)seg_c[seg] + all);
        }
      } else if (own) {
        if (IS_Q) qval[at] = 0.f;
        else cand[at].x = 0u;
      }
    }
    __syncwarp();
    for (int sg = lane; sg < a.n_seg; sg += 32) z += (double)seg_a[sg];
    Z = warp_sum(z);
    theta = th;
    n_ge = s.n - s.cum - less_at;
    return true;
  };

  // One thread: the predictor of a kind of row after a row (ok: theta found exactly).
  auto learn = [&](int kind, bool ok, int reason, float theta, float pivot, int n, int n_ge) {
    Predictor pr = sm.pred[kind];
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
      if (!rho_ok) {   // no usable density yet: stay in bootstrap mode
        pr.have = 0;
      } else {
        pr.theta = pr.have ? pr.theta + 0.25f * (theta - pr.theta) : theta;
        pr.rho = rho;
        pr.have = 1;
        // the next row's pivot: `margin` entries' worth below the predicted threshold; its
        // histogram spans three times that distance
        const float d = (float)a.margin / rho;
        pr.pivot = pr.theta - d;
        pr.inv_w = (float)kHistBins / (3.0f * d);
      }
    }
    sm.pred[kind] = pr;
  };

  auto reset_state = [&]() {   // all threads; nobody may be reading the selection scratch
    if (tid == 0) {
      rs.n_cand = 0;
      rs.n_member = 0;
      rs.overflow = 0;
      rs.max_key = 0;
      rs.alloc = 0;
    }
    if (tid < kHistBins) rs.hist[tid] = 0;
  };

  // Thread 0: leaves position g to the dense routines.
  auto defer = [&](size_t g) {
    const unsigned at = atomicAdd(a.dev_status + kFailCount, 1u);
    a.fail_list[at] = (int32_t)g;
    atomicAdd(a.dev_status + kCntRows, 1u);
  };

  // Two threads of different warps: the uniforms of a target position (`part` 0) and the
  // logit of x~ there (`part` 1).
  auto prepare_row = [&](RowPrep& pp, int child, int part) {
    const int t = (sm.ca * P.r + child / P.r) * P.W + sm.cc * P.r + child % P.r;
    const size_t g = (size_t)sm.b * P.H * P.W + t;
    if (part == 0) {
      const uint4 r = philox4x32_10(make_uint4((uint32_t)t, (uint32_t)sm.b + P.image_offset, P.round, 0u),
                                    make_uint2(P.seed_lo, P.seed_hi));
      pp.rnd[0] = r.x;
      pp.rnd[1] = r.y;
      pp.rnd[2] = r.z;
      return;
    }
    RowSrc tr = {a.cond + g * (size_t)P.V * esz, HAS_U ? a.uncond + g * (size_t)P.V * esz : nullptr, P.cfg_scale,
                 P.invT, P.V, BF16};
    pp.z_tok = load1(tr, sm.tok);
  };

  // Eq. 3-4 for the target row at position g, after its theta, m and Z_p are known (all threads;
  // four block barriers).  c_j = sum_{i<=j} p(n_i) along the neighbour list of x~; the leading
  // run with c_j < delta is pooled: J entries, mass c_J.  Leaves a bitmap of the pooled token ids
  // in the (by now unused) selection scratch of the row.
  auto pool_phase = [&](float theta, float m, double Zp, size_t g, double& cJ, int& J) {
    const int nb = P.pool_k - 1;
    const uint16_t* row = a.nn + (size_t)sm.tok * P.pool_k;
    uint32_t* const bitmap = reinterpret_cast<uint32_t*>(&rs);
    static_assert(sizeof(RowState::hist) + sizeof(RowState::member_z) + sizeof(RowState::member_at) +
                      sizeof(RowState::member_seg) >= 16384 / 8,
                  "the bitmap of a 16384-entry vocabulary must fit the selection scratch");
    const RowSrc tr = {a.cond + g * (size_t)P.V * esz, HAS_U ? a.uncond + g * (size_t)P.V * esz : nullptr,
                       P.cfg_scale, P.invT, P.V, BF16};
    __syncthreads();   // every warp is done with the set-aside entries
    for (int x = tid; x < (P.V + 31) / 32; x += kSThreads) bitmap[x] = 0u;
    if (tid == 0) {
      sm.first_bad = nb;
      sm.cJ = 0.0;
    }
    constexpr int PER = 8;   // list entries per thread: pool_k <= 2048
    const int per = (nb + kSThreads - 1) / kSThreads;
    const int j0 = tid * per;
    double loc[PER];
    int ids[PER];
    double run = 0.0;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      ids[i] = -1;
      loc[i] = run;
      if (i < per && j0 + i < nb) {
        int id = row[j0 + i + 1];
        if (id >= P.V) {
          atomicOr(a.dev_status, MULO_DEV_BAD_TOKEN);
          id = P.V - 1;
        }
        ids[i] = id;
        const float z = load1(tr, id);
        run += (z >= theta) ? (double)expf(__fsub_rn(z, m)) / Zp : 0.0;
        loc[i] = run;
      }
    }
    double inc = run;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double v = __shfl_up_sync(kFull, inc, o);
      if (lane >= o) inc += v;
    }
    if (lane == 31) sm.wsum[warp] = inc;
    // mass before this thread's entries: the lanes below (taken from the scan, not as inc - run: a
    // large entry in `run` would cancel the small masses before it), then the warps below
    double carry = __shfl_up_sync(kFull, inc, 1);
    if (lane == 0) carry = 0.0;
    __syncthreads();
    {
      double below = 0.0;
      for (int w = 0; w < warp; ++w) below += sm.wsum[w];
      carry = below + carry;
    }
    int bad = nb;
#pragma unroll
    for (int i = PER - 1; i >= 0; --i)
      if (ids[i] >= 0 && !(carry + loc[i] < P.pool_delta)) bad = j0 + i;
    if (bad < nb) atomicMin(&sm.first_bad, bad);
    __syncthreads();
    J = sm.first_bad;
#pragma unroll
    for (int i = 0; i < PER; ++i)
      if (ids[i] >= 0 && j0 + i < J) {
        atomicOr(&bitmap[ids[i] >> 5], 1u << (ids[i] & 31));
        if (j0 + i == J - 1) sm.cJ = carry + loc[i];
      }
    __syncthreads();
    cJ = sm.cJ;
  };

  // One thread, a phase ahead of prepare_row: asks L2 for the lines that hold the logit of x~ at
  // the next target position, so that the load there does not wait on HBM.
  auto prefetch_row = [&](int child) {
    const int t = (sm.ca * P.r + child / P.r) * P.W + sm.cc * P.r + child % P.r;
    const size_t off = (((size_t)sm.b * P.H * P.W + t) * (size_t)P.V + (size_t)sm.tok) * esz;
    asm volatile("prefetch.global.L2 [%0];" ::"l"(a.cond + off));
    if (HAS_U) asm volatile("prefetch.global.L2 [%0];" ::"l"(a.uncond + off));
  };

  for (int parent = p_begin; parent < p_end; ++parent) {
    // ------------------------------------------------------------ draft row
    {
      if (tid == 0) {
        if (!SAMPLE) sm.tok = checked_token(a.draft_tok_lo[parent], P.V, a.dev_status);
        // row addresses two parents ahead
        const int tp = sm.tparent + 1;
        if (parent > p_begin && tp < p_end) {
          int tb = sm.tb, tca = sm.tca, tcc = sm.tcc;
          if (++tcc == P.w) {
            tcc = 0;
            if (++tca == P.h) {
              tca = 0;
              ++tb;
            }
          }
          table_fill(a, sm, (tp - p_begin) & (kTableParents - 1), tp, tb, tca, tcc, esz);
          sm.tb = tb;
          sm.tca = tca;
          sm.tcc = tcc;
          sm.tparent = tp;
        }
      }
      float pivot, inv_w;
      choose_pivot(0, std::false_type{}, pivot, inv_w);
      stream_row(std::true_type{}, std::false_type{}, pivot, inv_w);
      __syncthreads();
      if (*(volatile int*)&sm.abort) {   // block-uniform: raised before the barrier
        // nothing more is written for this CTA's rows; its copies in flight (at most kStages chunks)
        // get a bounded time to land before the shared memory is given up
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        return;
      }
      if (!SAMPLE && tid == 64) prefetch_row(0);
      Sel s;
      bool ok = locate_bin(s);
      float theta = 0.f;
      int n_ge = 0;
      double Zq = 1.0;
      if (ok) exp_pass(std::true_type{}, s, pivot, inv_w);
      __syncthreads();
      if (ok) ok = finish_selection(std::true_type{}, s, theta, n_ge, Zq);
      if (tid == 0) {
        learn(0, ok, s.reason, theta, pivot, s.n, n_ge);
        sm.q_ok = ok;
        if (SAMPLE) {
          if (!ok) {
            atomicOr(a.dev_status, MULO_DEV_DENSE_FALLBACK);
            defer((size_t)parent);
          }
        } else if (ok) {
          // same rounding of Z_q as the unfused path (fp32 hi + lo)
          const float Zhi = (float)Zq, Zlo = (float)(Zq - (double)Zhi);
          const double Z = (double)Zhi + (double)Zlo;
          RowSrc qr = {a.draft + (size_t)parent * P.V * esz, nullptr, 0.f, P.invT, P.V, BF16};
          const float zq_tok = load1(qr, sm.tok);
          const double q = (zq_tok >= theta) ? exp((double)zq_tok - (double)s.m) / Z : 0.0;
          if (q <= 0.0) atomicOr(a.dev_status, MULO_DEV_ZERO_DRAFT_PROB);
          sm.theta_q = theta;
          sm.m_q = s.m;
          sm.Zq = Z;
          sm.q_tok = q;
          sm.invZq = (float)(1.0 / Z);
        } else {
          atomicOr(a.dev_status, MULO_DEV_DENSE_FALLBACK);
          for (int child = 0; child < rr; ++child)
            defer((size_t)sm.b * P.H * P.W + (sm.ca * P.r + child / P.r) * P.W + sm.cc * P.r + child % P.r);
        }
      }
      __syncthreads();   // everybody is done with the selection scratch
      reset_state();
      if (!SAMPLE && (tid == 64 || tid == 96) && ok)
        prepare_row(sm.prep[rowi & 1], 0, tid == 96);   // first child's uniforms and logit of x~
      if (SAMPLE && ok && warp == 0) {
        // y~ ~ q: inverse CDF over the row's candidate list (e = 0 below theta_q), then the token
        // id of the chosen entry from the look-up table of its segment
        const uint4 rnd = philox4x32_10(
            make_uint4((uint32_t)(sm.ca * P.w + sm.cc), (uint32_t)sm.b + P.image_offset, P.round, 1u),
            make_uint2(P.seed_lo, P.seed_hi));
        int sidx = 0;
        const int at = warp_draw(seg_c, a.n_seg, qseg, uniform24(rnd.x), [&](int i) { return qval[i]; }, &sidx);
        int tok = -1;
        if (at >= 0) {
          const int local = at - (int)qseg[sidx].x;   // rank of the entry within its segment
          const int cell0 = ((sidx / kSWarps) * a.chunk + (sidx % kSWarps) * SEG) / EPL;
          int found = -1;
          for (int k = lane; k < SEG / EPL; k += 32) {
            const unsigned cell = (cell0 + k) * EPL < P.V ? qcell[cell0 + k] : 0u;
            const unsigned m8 = cell & 0xffu;
            const int off = (int)(cell >> 8);
            if (m8 && off <= local && local < off + __popc(m8))
              found = (cell0 + k) * EPL + (int)__fns(m8, 0, local - off + 1);
          }
          const unsigned who = __ballot_sync(kFull, found >= 0);
          if (who) tok = __shfl_sync(kFull, found, __ffs(who) - 1);
        }
        if (lane == 0) a.sample_out[parent] = tok;
      }
      __syncthreads();
    }
    if (SAMPLE) {
      if (tid == 0) {   // next cell's coordinates (made visible by the barriers of its row)
        if (++sm.cc == P.w) {
          sm.cc = 0;
          if (++sm.ca == P.h) {
            sm.ca = 0;
            ++sm.b;
          }
        }
      }
      continue;
    }

    // ------------------------------------------------------------ children
    if (!sm.q_ok) {   // block-uniform: the whole parent went to the dense routines
      for (int child = 0; child < rr; ++child) skip_row();
      __syncthreads();
    } else {
      for (int child = 0; child < rr; ++child) {
        const RowPrep& pp = sm.prep[rowi & 1];
        float pivot, inv_w;
        choose_pivot(1, std::integral_constant<bool, HAS_U>{}, pivot, inv_w);
        stream_row(std::false_type{}, std::integral_constant<bool, HAS_U>{}, pivot, inv_w);
        __syncthreads();
        if (tid == 64 && child + 1 < rr) prefetch_row(child + 1);
        Sel s;
        bool ok = locate_bin(s);
        if (ok) {
          if (tid == 32) sm.e_tok = exp((double)pp.z_tok - (double)s.m);
          exp_pass(std::false_type{}, s, pivot, inv_w);
        }
        __syncthreads();
        float theta = 0.f;
        int n_ge = 0;
        double Zp = 1.0;
        if (ok) ok = finish_selection(std::false_type{}, s, theta, n_ge, Zp);
        const bool ok_sel = ok;   // the predictor learns from it while the draws run
        const int t = (sm.ca * P.r + child / P.r) * P.W + sm.cc * P.r + child % P.r;
        const size_t g = (size_t)sm.b * P.H * P.W + t;
        double cJ = 0.0;   // pooled mass of the neighbours of x~ (Eq. 3-4), J of them
        int J = 0;
        if constexpr (POOL) {
          if (ok) {   // block-uniform
            pool_phase(theta, s.m, Zp, g, cJ, J);
          }
        }
        const bool pooled = POOL && ok && J > 0;
        int draws = 0;
        float invZp = 0.f, invZq = 0.f;
        double mass = 0.0;   // P of Eq. 3: own probability plus pooled mass
        if (ok) {
          // ---- the decision (Eq. 1 / Eq. 5), the same in every warp
          const double e_tok = (pp.z_tok >= theta) ? sm.e_tok : 0.0;
          const double q_tok = sm.q_tok;
          int accepted;
          if (pooled) {
            mass = e_tok / Zp + cJ;
            if (P.accept_mode == MULO_ACCEPT_THRESHOLD) accepted = mass >= P.tau;
            else if (q_tok <= 0.0) accepted = mass > 0.0;
            else accepted = uniform24(pp.rnd[0]) < fmin(1.0, mass / q_tok);
          } else if (P.accept_mode == MULO_ACCEPT_THRESHOLD) accepted = e_tok >= P.tau * Zp;
          else if (q_tok <= 0.0) accepted = e_tok > 0.0;
          else accepted = uniform24(pp.rnd[0]) * q_tok * Zp < e_tok;
          draws = draws_for(P.resample_mode, accepted);
          invZp = 1.0f / (float)Zp;
          invZq = sm.invZq;
          if (tid == 0) {
            a.flags[g] = accepted ? 0 : 1;
            if (a.p_tok) a.p_tok[g] = (float)(e_tok / Zp);
            if (a.q_tok) a.q_tok[g] = (float)q_tok;
            if (a.accept_prob) {
              const double p = pooled ? mass : e_tok / Zp;
              double thr;
              if (P.accept_mode == MULO_ACCEPT_THRESHOLD) thr = p;
              else if (q_tok <= 0.0) thr = p > 0.0 ? 1.0 : 0.0;
              else thr = fmin(1.0, p / q_tok);
              a.accept_prob[g] = (float)thr;
            }
          }
        } else if (tid == 0) {
          atomicOr(a.dev_status, MULO_DEV_DENSE_FALLBACK);
          defer(g);
        }
        // weight of candidate i in the residual of Eq. 2 (lambda = 1)
        // (every token id of a target segment lies in the draft row's segment of the same
        // number, whose run starts at entry `qfirst` of the draft list)
        auto w_entry = [&](unsigned ebits, unsigned idbits, int qfirst) {
          const float pe = __fmul_rn(__uint_as_float(ebits), invZp);
          const int id = (int)idbits;
          const unsigned cell = qcell[id / EPL];
          const int j = id % EPL;
          float qe = 0.f;
          if ((cell >> j) & 1u) qe = qval[qfirst + (int)(cell >> 8) + __popc(cell & ((1u << j) - 1u))];
          return fmaxf(__fsub_rn(pe, __fmul_rn(qe, invZq)), 0.f);
        };
        auto w_resid = [&](int i) {
          const uint2 en = cand[i];
          return w_entry(en.x, en.y, (int)qseg[(int)en.y / SEG].x);
        };
        auto w_pair = [&](ushort2 r, int sl, int qfirst) {
          const uint4 v = *reinterpret_cast<const uint4*>(cand + r.x + sl);
          float w = w_entry(v.x, v.y, qfirst);
          if (sl + 1 < r.y) w += w_entry(v.z, v.w, qfirst);
          return w;
        };
        auto w_target = [&](int i) { return __uint_as_float(cand[i].x); };
        if (pooled) {   // block-uniform
          // p' in place: the pooled neighbours lose their mass, x~ gets P; the per-segment sums of
          // p' (target draw, and the fallback of a residual without mass) and of the residual
          const uint32_t* const bitmap = reinterpret_cast<const uint32_t*>(&rs);
          const unsigned e_pool = __float_as_uint((float)(mass * Zp));
          const int tok = sm.tok;
          for (int c0 = 0; c0 < a.n_chunks; c0 += groups) {
            const int c = c0 + grp;
            const bool has = c < a.n_chunks;
            const int seg = c * kSWarps + warp;
            float acc_b = 0.f, acc_c = 0.f;
            if (has) {
              const ushort2 r = tseg[seg];
              const int qfirst = qseg[seg].x;
              for (int sl = sub; sl < (int)r.y; sl += seg_lanes) {
                uint2 en = cand[r.x + sl];
                const int id = (int)en.y;
                if (id == tok) en.x = e_pool;
                else if ((bitmap[id >> 5] >> (id & 31)) & 1u) en.x = 0u;
                cand[r.x + sl].x = en.x;
                acc_c += __uint_as_float(en.x);
                if (draws & kDrawResidual) acc_b += w_entry(en.x, en.y, qfirst);
              }
            }
            __syncwarp();
            acc_b = seg_lanes_sum(acc_b, seg_lanes);
            acc_c = seg_lanes_sum(acc_c, seg_lanes);
            if (sub == 0 && has) {
              seg_b[seg] = acc_b;
              seg_c[seg] = acc_c;
            }
          }
        } else if (draws & kDrawResidual) {   // block-uniform
          for (int c0 = 0; c0 < a.n_chunks; c0 += groups) {
            const int c = c0 + grp;
            const bool has = c < a.n_chunks;
            const int seg = c * kSWarps + warp;
            float acc = 0.f;
            if (has) {
              const ushort2 r = tseg[seg];
              const int qfirst = qseg[seg].x;
              for (int sl = 2 * sub; sl < (int)r.y; sl += 4 * seg_lanes) {
                acc += w_pair(r, sl, qfirst);
                if (sl + 2 * seg_lanes < (int)r.y) acc += w_pair(r, sl + 2 * seg_lanes, qfirst);
              }
            }
            __syncwarp();
            acc = seg_lanes_sum(acc, seg_lanes);
            if (sub == 0 && has) seg_b[seg] = acc;
          }
        }
        __syncthreads();
        reset_state();
        if (ok && warp < 2) {
          // warp 0: the draw from the residual (a residual without mass falls back to the target
          // weights with the same uniform); warp 1: the draw from the target distribution.  Both
          // run the same code, the weight function picked at run time.
          int t_out = -1;
          if (draws & (warp == 0 ? kDrawResidual : kDrawTarget)) {
            bool resid = warp == 0;
            const double u = uniform24(pp.rnd[warp == 0 ? 1 : 2]);
#pragma unroll 1
            for (int attempt = 0; attempt < 2; ++attempt) {
              const int at = warp_draw(resid ? seg_b : seg_c, a.n_seg, tseg, u,
                                       [&](int i) { return resid ? w_resid(i) : w_target(i); });
              if (at >= 0) {
                t_out = (int)cand[at].y;
                break;
              }
              if (!resid) break;
              resid = false;
            }
          }
          if (lane == 0) (warp == 0 ? a.cand_res : a.cand_tgt)[g] = t_out;
        }
        if ((tid == 64 || tid == 96) && child + 1 < rr) prepare_row(sm.prep[(rowi + 1) & 1], child + 1, tid == 96);
        if (tid == 128) learn(1, ok_sel, s.reason, theta, pivot, s.n, n_ge);
        ++rowi;
        __syncthreads();
      }
    }
    // next parent's coordinates (made visible by the barriers of its draft row)
    if (tid == 0) {
      if (++sm.cc == P.w) {
        sm.cc = 0;
        if (++sm.ca == P.h) {
          sm.ca = 0;
          ++sm.b;
        }
      }
    }
  }
}

}  // namespace mulo
