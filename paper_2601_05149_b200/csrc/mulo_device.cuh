// Device-side building blocks shared by the MuLo-SD kernels: logit
// pre-processing, Philox4x32-10, block reductions/scans, and the "dense" row
// routines that work on a whole vocabulary row straight from global memory.
//
// The dense routines are the general path: any V (multiple of 8), top-k on or
// off, fp32 or bf16 logits.  They read a row several times (it stays in L1/L2
// after the first read) and are what the fast top-k path falls back to.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace mulo {

constexpr int kThreads = 512;           // threads per CTA of the row kernels
constexpr int kWarps = kThreads / 32;
constexpr unsigned kFull = 0xffffffffu;

// ------------------------------------------------------------------ Philox
// Philox4x32 with 10 rounds (Salmon et al., SC'11).  Counter (position, image,
// round, tag), key (seed low, seed high).
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint32_t a = 0xD2511F53u, b = 0xCD9E8D57u;
    uint32_t h0 = __umulhi(a, c.x), l0 = a * c.x;
    uint32_t h1 = __umulhi(b, c.z), l1 = b * c.z;
    c = make_uint4(h1 ^ c.y ^ k.x, l1, h0 ^ c.w ^ k.y, l0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}

// top 24 bits of a word as a uniform in [0,1): exact in fp32 and fp64
__device__ __forceinline__ double uniform24(uint32_t w) { return (double)(w >> 8) * (1.0 / 16777216.0); }

// ------------------------------------------------------- logits -> z (fp32)
// The three roundings below ARE the definition of a pre-processed logit:
//   d = c - u;  v = fma(s, d, u);  z = v * invT        (IEEE fp32, round-to-nearest)
// Written with _rn intrinsics so the compiler can neither fuse nor reorder them.
__device__ __forceinline__ float mix_logit(float c, float u, bool has_u, float s, float invT) {
  float v = c;
  if (has_u) v = __fmaf_rn(s, __fsub_rn(c, u), u);
  return __fmul_rn(v, invT);
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

struct RowSrc {          // one vocabulary row in global memory
  const char* cond;      // conditional (or the only) logits of the row
  const char* uncond;    // unconditional logits, or nullptr
  float s, invT;
  int V;
  int bf16;
};

// eight consecutive pre-processed logits starting at x (x % 8 == 0)
__device__ __forceinline__ void load8(const RowSrc& r, int x, float (&z)[8]) {
  const bool hu = r.uncond != nullptr;
  if (r.bf16) {
    uint4 c = __ldg(reinterpret_cast<const uint4*>(r.cond + (size_t)x * 2));
    uint4 u = make_uint4(0, 0, 0, 0);
    if (hu) u = __ldg(reinterpret_cast<const uint4*>(r.uncond + (size_t)x * 2));
    z[0] = mix_logit(bf16_lo(c.x), bf16_lo(u.x), hu, r.s, r.invT);
    z[1] = mix_logit(bf16_hi(c.x), bf16_hi(u.x), hu, r.s, r.invT);
    z[2] = mix_logit(bf16_lo(c.y), bf16_lo(u.y), hu, r.s, r.invT);
    z[3] = mix_logit(bf16_hi(c.y), bf16_hi(u.y), hu, r.s, r.invT);
    z[4] = mix_logit(bf16_lo(c.z), bf16_lo(u.z), hu, r.s, r.invT);
    z[5] = mix_logit(bf16_hi(c.z), bf16_hi(u.z), hu, r.s, r.invT);
    z[6] = mix_logit(bf16_lo(c.w), bf16_lo(u.w), hu, r.s, r.invT);
    z[7] = mix_logit(bf16_hi(c.w), bf16_hi(u.w), hu, r.s, r.invT);
  } else {
    const float4* cp = reinterpret_cast<const float4*>(r.cond + (size_t)x * 4);
    float4 c0 = __ldg(cp), c1 = __ldg(cp + 1);
    float4 u0 = make_float4(0, 0, 0, 0), u1 = u0;
    if (hu) {
      const float4* up = reinterpret_cast<const float4*>(r.uncond + (size_t)x * 4);
      u0 = __ldg(up);
      u1 = __ldg(up + 1);
    }
    z[0] = mix_logit(c0.x, u0.x, hu, r.s, r.invT);
    z[1] = mix_logit(c0.y, u0.y, hu, r.s, r.invT);
    z[2] = mix_logit(c0.z, u0.z, hu, r.s, r.invT);
    z[3] = mix_logit(c0.w, u0.w, hu, r.s, r.invT);
    z[4] = mix_logit(c1.x, u1.x, hu, r.s, r.invT);
    z[5] = mix_logit(c1.y, u1.y, hu, r.s, r.invT);
    z[6] = mix_logit(c1.z, u1.z, hu, r.s, r.invT);
    z[7] = mix_logit(c1.w, u1.w, hu, r.s, r.invT);
  }
}

// one pre-processed logit (gather)
__device__ __forceinline__ float load1(const RowSrc& r, int x) {
  const bool hu = r.uncond != nullptr;
  float c, u = 0.f;
  if (r.bf16) {
    c = __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(r.cond) + x) << 16);
    if (hu) u = __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(r.uncond) + x) << 16);
  } else {
    c = __ldg(reinterpret_cast<const float*>(r.cond) + x);
    if (hu) u = __ldg(reinterpret_cast<const float*>(r.uncond) + x);
  }
  return mix_logit(c, u, hu, r.s, r.invT);
}

// order-preserving map float -> uint32 (-0 and +0 map to the same key)
__device__ __forceinline__ uint32_t float_key(float f) {
  uint32_t b = __float_as_uint(f + 0.0f);
  return b ^ ((b & 0x80000000u) ? 0xffffffffu : 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k) {
  uint32_t b = (k & 0x80000000u) ? (k ^ 0x80000000u) : ~k;
  return __uint_as_float(b);
}

// ------------------------------------------------------ block-wide helpers
struct BlockScratch {
  double d[kWarps];
  float f[kWarps];
  double ex[kThreads + 1];
  unsigned hist[256];
  unsigned sel_digit, sel_k;
  int owner;
  int found;
  int bi[8];
  double bd[8];
};

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}

// every thread receives the same total (fixed summation order)
__device__ __forceinline__ double block_sum(double v, BlockScratch& bs) {
  v = warp_sum(v);
  if ((threadIdx.x & 31) == 0) bs.d[threadIdx.x >> 5] = v;
  __syncthreads();
  double t = 0.0;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) t += bs.d[w];
  __syncthreads();
  return t;
}

__device__ __forceinline__ float block_max(float v, BlockScratch& bs) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, o));
  if ((threadIdx.x & 31) == 0) bs.f[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = bs.f[0];
#pragma unroll
  for (int w = 1; w < kWarps; ++w) t = fmaxf(t, bs.f[w]);
  __syncthreads();
  return t;
}

// exclusive prefix sums of one value per thread into bs.ex[0..kThreads]
// (bs.ex[kThreads] = total).  Ends with a barrier.
__device__ __forceinline__ void block_exscan(double v, BlockScratch& bs) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    double n = __shfl_up_sync(kFull, inc, o);
    if (lane >= o) inc += n;
  }
  double exc = __shfl_up_sync(kFull, inc, 1);
  if (lane == 0) exc = 0.0;
  if (lane == 31) bs.d[warp] = inc;
  __syncthreads();
  double pre = 0.0;
  for (int w = 0; w < warp; ++w) pre += bs.d[w];
  bs.ex[threadIdx.x] = pre + exc;
  if (threadIdx.x == kThreads - 1) bs.ex[kThreads] = pre + inc;
  __syncthreads();
}

// elements [beg, end) of a row owned by this thread in the dense routines:
// contiguous runs of E (a multiple of 8, the same for every thread), so that a
// per-thread sum is a slice of the ascending-id CDF.  Runs past the row's end
// are empty; loops that use warp collectives iterate all E/8 chunks and test
// `x < V` per chunk so that every lane of a warp makes the same trips.
__device__ __forceinline__ int dense_run(int V) { return 8 * ((V + 8 * kThreads - 1) / (8 * kThreads)); }

// ------------------------------------------------ dense: top-k, max, sum
// theta = value of the top_k-th largest pre-processed logit (-inf when top-k
// is off), m = row maximum, Z = sum over {z >= theta} of exp(z - m).
// All threads return the same values.
__device__ inline void dense_row_stats(const RowSrc& r, int top_k, BlockScratch& bs, float& theta,
                                       float& m, double& Z) {
  const int E = dense_run(r.V);
  const int beg = (int)threadIdx.x * E;
  const int end = min(r.V, beg + E);
  float z[8];
  float mx = -INFINITY;
  for (int x = beg; x < end; x += 8) {
    load8(r, x, z);
#pragma unroll
    for (int j = 0; j < 8; ++j) mx = fmaxf(mx, z[j]);
  }
  m = block_max(mx, bs);
  theta = -INFINITY;
  if (top_k > 0 && top_k < r.V) {
    // MSB-first radix select on order-preserving keys, 8 bits per pass
    uint32_t prefix = 0, mask = 0;
    unsigned kk = (unsigned)top_k;
    for (int shift = 24; shift >= 0; shift -= 8) {
      if (threadIdx.x < 256) bs.hist[threadIdx.x] = 0;
      __syncthreads();
      for (int x = beg; x < beg + E; x += 8) {
        const bool valid = x < r.V;
        if (valid) load8(r, x, z);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          uint32_t key = float_key(z[j]);
          bool in = valid && (key & mask) == prefix;
          uint32_t digit = (key >> shift) & 255u;
          // warp-aggregated histogram update: one atomic per distinct digit
          unsigned act = __ballot_sync(kFull, in);
          if (in) {
            unsigned peers = __match_any_sync(act, digit);
            if ((int)(threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&bs.hist[digit], __popc(peers));
          }
        }
      }
      __syncthreads();
      if (threadIdx.x == 0) {
        unsigned cum = 0;
        int dgt = 255;
        for (; dgt > 0; --dgt) {
          if (cum + bs.hist[dgt] >= kk) break;
          cum += bs.hist[dgt];
        }
        bs.sel_digit = (unsigned)dgt;
        bs.sel_k = kk - cum;
      }
      __syncthreads();
      prefix |= bs.sel_digit << shift;
      mask |= 255u << shift;
      kk = bs.sel_k;
      __syncthreads();
    }
    theta = key_float(prefix);
  }
  double acc = 0.0;
  for (int x = beg; x < end; x += 8) {
    load8(r, x, z);
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (z[j] >= theta) acc += (double)expf(__fsub_rn(z[j], m));
  }
  Z = block_sum(acc, bs);
}

}  // namespace mulo
