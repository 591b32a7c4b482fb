/*
 * mulo_oracle.c -- plain CPU statement of the MuLo-SD draft-and-verify round.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is the slow, obviously-correct
 * restatement of what the CUDA library computes; the tests, the smoke check and
 * the CPU-baseline leg of the benchmark are its only callers.  It shares no
 * code, header, table or helper with the CUDA path and the product never calls
 * it.  Everything after the fp32 logit pre-processing is double precision,
 * loops are sequential and in the order the paper's definitions are written.
 *
 * Passages followed (paper: "Multi-Scale Local Speculative Decoding for Image
 * Generation"):
 *   Sec. 3.1 Eq. 1   acceptance  u < min(1, p(x~)/q(x~))
 *   Sec. 3.1 Eq. 2   residual    norm(max(0, p - q))
 *   Sec. 3.1 Eq. 3   pooled numerator  sum_{x in B_k(x~)} p(x)
 *   Sec. 3.1 Eq. 4   TVD(p^(k,delta), p) < delta, mass moved inside A_{k,delta}
 *   Sec. 3.2 Step 2  x~ = U_r(y~): sequence length grows by r^2
 *   Sec. 3.3 Eq. 5   relaxed rule: accept iff pooled mass >= tau
 *   Sec. 3.3 Eq. 6   N(t,l) = {u : |i_u-i_t|<=l, |j_u-j_t|<=l, u >= t_0}
 *   Sec. 3.3 Eq. 7   R_X = union of N(t,l) over rejected t
 *   Algorithm 1      Step 4 (accept), Step 5 (expand), Step 6 (resample from M_p)
 *   Sec. 3.4 Eq. 8   rejection islands {I_m} = CC_8(R_X): 8-connected components
 *   Sec. 3.4         island-parallel redraw with a ZipAR-style row window: step index
 *   Sec. 3.2 Step 1  y~ ~ M_q: the drafter's own sampling, on given logits
 *   Sec. 3.2 Step 7  y = D_r(x): stand-in, majority token of each r x r block
 *   Supp. "Sampling" temperature, top-k, classifier-free guidance of the sampler
 *
 * Readings taken where the paper is silent (each is listed in the design notes):
 *   - U_r stand-in: nearest-neighbour replication of the low-res token AND of
 *     the low-res draft distribution (integer division of coordinates by r).
 *   - logits -> probabilities:  CFG mix, then * 1/T, then top-k mask, then
 *     softmax.  The first three steps are IEEE fp32 operations in exactly this
 *     order (d = c - u; z = fmaf(s, d, u); z = z * invT) so that the top-k set
 *     is a well defined function of the inputs.  Top-k keeps every entry whose
 *     value is >= the k-th largest value (ties kept).
 *   - A_{k,delta}: longest prefix n_1..n_J of the distance-sorted neighbour
 *     list whose added target mass c_J stays < delta; pooled mass
 *     P = p(x~) + c_J; p' moves that mass onto x~.
 *   - uniforms: Philox4x32-10, key = (seed lo, seed hi), counter =
 *     (position, image, round, tag); word 0 -> acceptance, word 1 -> residual
 *     draw, word 2 -> target draw; u = (word >> 8) * 2^-24.
 *   - positions of R_X that were individually accepted are redrawn from p'
 *     (Algorithm 1 Step 6), rejected ones from the residual (Eq. 2), unless a
 *     mode flag forces one rule for all.  A fourth mode uses the residual only
 *     for a rejected position that no OTHER rejection would have swept in (none
 *     in its window, or it is the image's first rejection and clipping is on)
 *     and p' everywhere else in R_X: with independent draft tokens that is the
 *     rule under which every output is distributed exactly as p for l > 0.
 *
 * Parity pins (tests/, CPU only): Philox known answers; softmax/top-k against
 * torch in fp64; target == draft accepts everything; E[accept] = sum min(p,q);
 * residual mass = TVD; exact output pmf by enumeration of all 2^24 uniforms;
 * chi-square of the whole round; dilation against scipy and brute force;
 * inverse CDF against numpy.searchsorted; islands against scipy.ndimage.label,
 * against reachability by boolean matrix closure on every mask of a small grid,
 * and on hand-drawn shapes; the draft sampler against the pinned primitives
 * composed in the test and by chi-square over rounds; the down-sampler by
 * D_r(U_r(y)) = y, scipy.stats.mode on blocks without ties, and hand-written
 * blocks with ties; the island schedule by a time-stepped simulation of the
 * rule, the closed form W + (H - 1) w of a full grid, and island size when the
 * window spans the row.  The paper prints no worked numeric example for this
 * path, so no pin is a printed value.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_F32 0
#define ORC_BF16 1

#define ORC_ACCEPT_RATIO 0
#define ORC_ACCEPT_THRESHOLD 1

#define ORC_RESAMPLE_MIXED 0
#define ORC_RESAMPLE_RESIDUAL_ALL 1
#define ORC_RESAMPLE_TARGET_ALL 2
#define ORC_RESAMPLE_ISOLATED_RESIDUAL 3

/* borderline flags reported per position */
#define ORC_FLAG_ACCEPT_EDGE 1u /* |u - thr| < 1e-6 (or pooled mass within 1e-6 rel. of tau) */
#define ORC_FLAG_CDF_EDGE 2u    /* u' within 1e-6 of an edge of the chosen bin of the normalised CDF,
                                   or a residual holding less than ORC_MIN_RESIDUAL_MASS      */
#define ORC_FLAG_POOL_EDGE 4u   /* some prefix mass c_j within 1e-6 of delta          */
#define ORC_MIN_RESIDUAL_MASS 1e-5

typedef struct {
  int32_t H, W, V, r;
  int32_t dtype;          /* ORC_F32 / ORC_BF16, all logit tensors                */
  float temperature;      /* > 0                                                  */
  int32_t top_k;          /* <= 0 or >= V: off                                    */
  float cfg_scale;        /* used iff an unconditional tensor is given            */
  int32_t accept_mode;    /* ORC_ACCEPT_*                                         */
  float tau;              /* Eq. 5 threshold                                      */
  int32_t pool_k;         /* <= 1: pooling off                                    */
  float pool_delta;       /* Eq. 4 bound                                          */
  int32_t radius;         /* l of Eq. 6                                           */
  int32_t clip_before_first; /* apply the "u >= t_0" clause of Eq. 6              */
  int32_t resample_mode;  /* ORC_RESAMPLE_*                                       */
  uint64_t seed;
  uint32_t round;
  uint32_t image;         /* global image index used in the Philox counter        */
} orc_params;

/* ------------------------------------------------------------------ Philox */

/* Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11): two 32x32->64
 * multiplies per round, the high words xor-ed with the other counter words and
 * the key, the key bumped by the Weyl constants between rounds. */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t prod0 = (uint64_t)M0 * c0;
    uint64_t prod1 = (uint64_t)M1 * c2;
    uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)prod0;
    uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)prod1;
    uint32_t n0 = hi1 ^ c1 ^ k0;
    uint32_t n1 = lo1;
    uint32_t n2 = hi0 ^ c3 ^ k1;
    uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += W0; k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* top 24 bits -> [0,1): exactly representable in fp32 and in double */
double orc_uniform24(uint32_t word) { return (double)(word >> 8) * (1.0 / 16777216.0); }

/* the three uniforms of one (seed, image, position, round): accept, residual, target */
void orc_position_uniforms(uint64_t seed, uint32_t image, uint32_t position, uint32_t round,
                           uint32_t tag, double u[3]) {
  uint32_t ctr[4] = {position, image, round, tag};
  uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
  uint32_t w[4];
  orc_philox4x32_10(ctr, key, w);
  u[0] = orc_uniform24(w[0]);
  u[1] = orc_uniform24(w[1]);
  u[2] = orc_uniform24(w[2]);
}

/* ------------------------------------------------------- logits -> z (fp32) */

static float load_logit(const void* base, int dtype, size_t idx) {
  if (dtype == ORC_BF16) {
    uint32_t bits = (uint32_t)((const uint16_t*)base)[idx] << 16; /* bf16 -> fp32 is exact */
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
  }
  return ((const float*)base)[idx];
}

/* One row of V pre-processed logits.  cond/uncond point at element 0 of the row
 * (uncond may be NULL).  The three fp32 roundings are the specification. */
void orc_preprocess_row(const void* cond, const void* uncond, int dtype, int V, float cfg_scale,
                        float temperature, float* z) {
  const float invT = 1.0f / temperature;
  for (int x = 0; x < V; ++x) {
    float c = load_logit(cond, dtype, (size_t)x);
    float v = c;
    if (uncond) {
      float un = load_logit(uncond, dtype, (size_t)x);
      float d = c - un;
      v = fmaf(cfg_scale, d, un); /* l = l_u + s (l_c - l_u) */
    }
    z[x] = v * invT;
  }
}

static int cmp_float_desc(const void* a, const void* b) {
  float fa = *(const float*)a, fb = *(const float*)b;
  return (fa < fb) - (fa > fb);
}

/* value of the top_k-th largest entry; -inf when top-k is off */
float orc_topk_threshold(const float* z, int V, int top_k) {
  if (top_k <= 0 || top_k >= V) return -INFINITY;
  float* sorted = (float*)malloc((size_t)V * sizeof(float));
  memcpy(sorted, z, (size_t)V * sizeof(float));
  qsort(sorted, (size_t)V, sizeof(float), cmp_float_desc);
  float theta = sorted[top_k - 1];
  free(sorted);
  return theta;
}

/* softmax over the entries with z >= theta, 0 elsewhere; returns max and sum */
void orc_softmax_masked(const float* z, int V, float theta, double* prob, double* m_out,
                        double* Z_out) {
  double m = -INFINITY;
  for (int x = 0; x < V; ++x)
    if (z[x] >= theta && (double)z[x] > m) m = (double)z[x];
  double Z = 0.0;
  for (int x = 0; x < V; ++x)
    if (z[x] >= theta) Z += exp((double)z[x] - m);
  for (int x = 0; x < V; ++x) prob[x] = (z[x] >= theta) ? exp((double)z[x] - m) / Z : 0.0;
  *m_out = m;
  *Z_out = Z;
}

/* ----------------------------------------------------------------- pooling */

/* Eq. 3-4.  nn_row = the pool_k ids nearest to tok in the codebook, entry 0 is
 * tok itself.  c_j = sum_{m=1..j} p(n_m); J = max{j >= 0 : c_j < delta} with
 * c_0 = 0, and J = 0 if delta <= 0.  Writes p' (a copy of p with the mass of
 * n_1..n_J moved onto tok) and returns P = p(tok) + c_J.  *gap = min_j |c_j -
 * delta| over j = 1..pool_k-1 (how close the choice of J was to flipping). */
double orc_pool(const double* p, int V, const uint16_t* nn_row, int pool_k, double delta, int tok,
                double* p_prime, int* J_out, double* gap) {
  memcpy(p_prime, p, (size_t)V * sizeof(double));
  *gap = INFINITY;
  if (pool_k <= 1 || nn_row == NULL) {
    *J_out = 0;
    return p[tok];
  }
  double c = 0.0, cJ = 0.0;
  int J = 0;
  int open = 1; /* prefix property: stop extending at the first c_j >= delta */
  for (int j = 1; j < pool_k; ++j) {
    c += p[nn_row[j]];
    double g = fabs(c - delta);
    if (g < *gap) *gap = g;
    if (open && c < delta) {
      J = j;
      cJ = c;
    } else {
      open = 0;
    }
  }
  for (int j = 1; j <= J; ++j) p_prime[nn_row[j]] = 0.0;
  double P = p[tok] + cJ;
  p_prime[tok] = P;
  *J_out = J;
  return P;
}

/* ------------------------------------------------------------- acceptance */

/* Eq. 1 with the pooled numerator of Eq. 3: min(1, P / q).  q == 0 cannot
 * happen for a token drawn from q; it is read as "accept iff P > 0". */
double orc_accept_threshold(double P, double q) {
  if (q <= 0.0) return P > 0.0 ? 1.0 : 0.0;
  double ratio = P / q;
  return ratio < 1.0 ? ratio : 1.0;
}

/* --------------------------------------------------------------- sampling */

/* Inverse CDF over weights w[0..V) in ascending token id with uniform u in
 * [0,1): token = min{x : C(x) > u * Z}, C(x) = sum_{x' <= x} w(x').  Returns -1
 * if Z == 0.  *edge_gap = distance (in units of the normalised CDF) from u to
 * the nearer edge of the chosen bin. */
int orc_inverse_cdf(const double* w, int V, double u, double* Z_out, double* edge_gap) {
  double Z = 0.0;
  for (int x = 0; x < V; ++x) Z += w[x];
  if (Z_out) *Z_out = Z;
  if (!(Z > 0.0)) {
    if (edge_gap) *edge_gap = INFINITY;
    return -1;
  }
  double y = u * Z;
  double C = 0.0;
  int chosen = -1;
  double lo = 0.0, hi = 0.0;
  for (int x = 0; x < V; ++x) {
    double before = C;
    C += w[x];
    if (C > y) {
      chosen = x;
      lo = before;
      hi = C;
      break;
    }
  }
  if (chosen < 0) { /* u*Z rounded up to the total: take the last token with weight */
    for (int x = V - 1; x >= 0; --x)
      if (w[x] > 0.0) {
        chosen = x;
        break;
      }
    lo = Z - w[chosen];
    hi = Z;
  }
  if (edge_gap) {
    double g0 = fabs(u - lo / Z), g1 = fabs(hi / Z - u);
    *edge_gap = g0 < g1 ? g0 : g1;
  }
  return chosen;
}

/* w(x) = max(0, p'(x) - lambda q(x))  (Eq. 2 for lambda = 1; p' itself for lambda = 0) */
void orc_residual_weights(const double* p_prime, const double* q, int V, double lambda, double* w) {
  for (int x = 0; x < V; ++x) {
    double d = p_prime[x] - lambda * q[x];
    w[x] = d > 0.0 ? d : 0.0;
  }
}

/* ------------------------------------------------------------------- masks */

/* Eq. 6-7 by the set definition.  reject/expand are H*W bytes (0/1).  Returns
 * t_0 = first rejected raster index, or H*W when nothing was rejected. */
int orc_expand(const uint8_t* reject, int H, int W, int radius, int clip_before_first,
               uint8_t* expand) {
  const int N = H * W;
  int t0 = N;
  if (H <= 0 || W <= 0) return 0;
  for (int t = 0; t < N; ++t)
    if (reject[t]) {
      t0 = t;
      break;
    }
  memset(expand, 0, (size_t)N);
  for (int t = 0; t < N; ++t) {
    if (!reject[t]) continue;
    int it = t / W, jt = t % W;
    for (int u = 0; u < N; ++u) {
      int iu = u / W, ju = u % W;
      if (abs(iu - it) <= radius && abs(ju - jt) <= radius && (!clip_before_first || u >= t0))
        expand[u] = 1;
    }
  }
  return t0;
}

/* Eq. 8: the rejection islands are the classes of R_X under "joined by a chain
 * of positions of R_X in which consecutive positions differ by at most 1 in
 * both coordinates".  Written out as that definition: walk the grid in raster
 * order; a position of R_X that has no island yet opens island m = M + 1 and
 * everything reachable from it through 8-neighbours gets m.  Islands are thereby
 * numbered by the raster index of their first position (a convention of this
 * code; the paper leaves the numbering open).
 *   in_rx   [H*W] bytes (0/1);  labels [H*W] out, 0 outside R_X;
 *   rows    [H*W][2] out: first and last grid row of islands 1..M (entry m-1);
 *   size    [H*W]    out: number of positions.   Returns M. */
int orc_islands(const uint8_t* in_rx, int H, int W, int32_t* labels, int32_t* rows, int32_t* size) {
  const int N = H * W;
  if (H <= 0 || W <= 0) return 0;
  int32_t* stack = (int32_t*)malloc(sizeof(int32_t) * (size_t)N);
  int M = 0;
  for (int t = 0; t < N; ++t) labels[t] = 0;
  for (int t = 0; t < N; ++t) {
    if (!in_rx[t] || labels[t]) continue;
    ++M;
    int top = 0;
    stack[top++] = t;
    labels[t] = M;
    rows[2 * (M - 1)] = t / W;
    rows[2 * (M - 1) + 1] = t / W;
    size[M - 1] = 0;
    while (top > 0) {
      const int v = stack[--top];
      const int iv = v / W, jv = v % W;
      size[M - 1] += 1;
      if (iv < rows[2 * (M - 1)]) rows[2 * (M - 1)] = iv;
      if (iv > rows[2 * (M - 1) + 1]) rows[2 * (M - 1) + 1] = iv;
      for (int di = -1; di <= 1; ++di)
        for (int dj = -1; dj <= 1; ++dj) {
          const int iu = iv + di, ju = jv + dj;
          if ((di == 0 && dj == 0) || iu < 0 || iu >= H || ju < 0 || ju >= W) continue;
          const int u = iu * W + ju;
          if (in_rx[u] && !labels[u]) {
            labels[u] = M;
            stack[top++] = u;
          }
        }
    }
  }
  free(stack);
  return M;
}

/* Sec. 3.4, "within each island the ZipAR decoding strategy": the sequential
 * target-model step at which each position of R_X is redrawn when the islands
 * run concurrently and, inside an island, rows advance left to right with the
 * row-window rule of ZipAR-w: a position may be decoded one step after its
 * predecessor in the same row of the island, and one step after the row above
 * (of the same island) has been decoded up to `window - 1` columns beyond it:
 *   step(t) = 1 + max( step(previous position of the island in row i),
 *                      max{ step(u) : u in the island, row(u) = i - 1,
 *                                     col(u) <= col(t) + window - 1 } ),
 * a maximum over nothing counting as 0.  (The paper names the strategy and the
 * window, 16; this recurrence is the reading taken for it.)
 *   labels [H*W] island numbers (0 outside R_X);  step [H*W] out, 0 outside R_X.
 * Returns the number of sequential steps of the image, max step. */
int orc_island_schedule(const int32_t* labels, int H, int W, int window, int32_t* step) {
  int nfe = 0;
  for (int i = 0; i < H; ++i)
    for (int j = 0; j < W; ++j) {
      const int m = labels[i * W + j];
      step[i * W + j] = 0;
      if (m <= 0) continue;
      int before = 0;
      for (int jj = 0; jj < j; ++jj) /* predecessor(s) in the same row */
        if (labels[i * W + jj] == m && step[i * W + jj] > before) before = step[i * W + jj];
      if (i > 0)
        for (int jj = 0; jj < W && jj <= j + window - 1; ++jj)
          if (labels[(i - 1) * W + jj] == m && step[(i - 1) * W + jj] > before)
            before = step[(i - 1) * W + jj];
      step[i * W + j] = before + 1;
      if (before + 1 > nfe) nfe = before + 1;
    }
  return nfe;
}

/* ---------------------------------------------------------------- stages */

/* Step 2 stand-in + draft statistics for ONE image.
 *   draft_lo   [h, w, V] logits, draft_tok_lo [h, w]
 *   tok_hi     [H, W]           up-sampled tokens
 *   stats_lo   [h, w, 3] double (theta_q, m_q, Z_q)
 *   q_tok_hi   [H, W]    double  q(x~) at every target position            */
void orc_upsample_pool_image(const orc_params* P, const void* draft_lo, const int32_t* draft_tok_lo,
                             int32_t* tok_hi, double* stats_lo, double* q_tok_hi) {
  const int H = P->H, W = P->W, V = P->V, r = P->r, h = H / r, w = W / r;
  const size_t esz = P->dtype == ORC_BF16 ? 2 : 4;
  float* z = (float*)malloc((size_t)V * sizeof(float));
  double* q = (double*)malloc((size_t)V * sizeof(double));
  double* q_tok_lo = (double*)malloc((size_t)h * w * sizeof(double));
  for (int a = 0; a < h; ++a)
    for (int c = 0; c < w; ++c) {
      const size_t cell = (size_t)a * w + c;
      const char* row = (const char*)draft_lo + cell * (size_t)V * esz;
      orc_preprocess_row(row, NULL, P->dtype, V, 0.0f, P->temperature, z);
      float theta = orc_topk_threshold(z, V, P->top_k);
      double m, Z;
      orc_softmax_masked(z, V, theta, q, &m, &Z);
      stats_lo[cell * 3 + 0] = (double)theta;
      stats_lo[cell * 3 + 1] = m;
      stats_lo[cell * 3 + 2] = Z;
      q_tok_lo[cell] = q[draft_tok_lo[cell]];
    }
  for (int i = 0; i < H; ++i)
    for (int j = 0; j < W; ++j) {
      const size_t cell = (size_t)(i / r) * w + (size_t)(j / r);
      tok_hi[(size_t)i * W + j] = draft_tok_lo[cell];
      q_tok_hi[(size_t)i * W + j] = q_tok_lo[cell];
    }
  free(z);
  free(q);
  free(q_tok_lo);
}

/* Everything that one visit of a target position computes, given the parent's
 * q row.  Returns the accept bit; fills the per-position records. */
typedef struct {
  double p_tok, q_tok, accept_prob;
  int accepted;
  uint32_t flags;
  int tok_residual, tok_target; /* inverse-CDF draws with lambda = 1 / lambda = 0 */
  uint32_t flag_residual, flag_target;
} orc_position;

static void visit_position(const orc_params* P, const float* zt, const double* q, int tok,
                           const uint16_t* nn, uint32_t position, double* p, double* p_prime,
                           double* wts, orc_position* out) {
  const int V = P->V;
  float theta = orc_topk_threshold(zt, V, P->top_k);
  double m, Z;
  orc_softmax_masked(zt, V, theta, p, &m, &Z);
  int J;
  double gap;
  const uint16_t* nn_row = (P->pool_k > 1 && nn) ? nn + (size_t)tok * P->pool_k : NULL;
  double mass = orc_pool(p, V, nn_row, P->pool_k, (double)P->pool_delta, tok, p_prime, &J, &gap);
  double u[3];
  orc_position_uniforms(P->seed, P->image, position, P->round, 0u, u);
  out->p_tok = p[tok];
  out->q_tok = q[tok];
  out->flags = 0;
  if (gap < 1e-6) out->flags |= ORC_FLAG_POOL_EDGE;
  if (P->accept_mode == ORC_ACCEPT_THRESHOLD) {
    /* Eq. 5: no q, no uniform */
    out->accept_prob = mass;
    out->accepted = mass >= (double)P->tau;
    if (fabs(mass - (double)P->tau) < 1e-6 * fabs((double)P->tau)) out->flags |= ORC_FLAG_ACCEPT_EDGE;
  } else {
    double thr = orc_accept_threshold(mass, q[tok]);
    out->accept_prob = thr;
    out->accepted = u[0] < thr;
    if (fabs(u[0] - thr) < 1e-6) out->flags |= ORC_FLAG_ACCEPT_EDGE;
  }
  /* both candidate draws: lambda = 1 (Eq. 2, uniform word 1) and lambda = 0
   * (Algorithm 1 Step 6, uniform word 2).  A residual without mass falls back
   * to the lambda = 0 weights but keeps its own uniform. */
  double Zw, eg;
  orc_residual_weights(p_prime, q, V, 1.0, wts);
  int t1 = orc_inverse_cdf(wts, V, u[1], &Zw, &eg);
  if (t1 < 0) {
    orc_residual_weights(p_prime, q, V, 0.0, wts);
    t1 = orc_inverse_cdf(wts, V, u[1], &Zw, &eg);
  }
  out->tok_residual = t1;
  /* A draw is borderline when its uniform lies within 1e-6 of an edge of the chosen bin of the
   * NORMALISED CDF.  One more case: a residual that holds less than ORC_MIN_RESIDUAL_MASS of
   * probability (target and draft all but equal) is rounding dust -- its shape is not defined
   * at the precision of the probabilities themselves -- so every draw from it is borderline.
   * (After the fall-back to the target weights Z_w = 1 and only the edge test applies.) */
  out->flag_residual = (eg < 1e-6 || Zw < ORC_MIN_RESIDUAL_MASS) ? ORC_FLAG_CDF_EDGE : 0u;
  orc_residual_weights(p_prime, q, V, 0.0, wts);
  int t0 = orc_inverse_cdf(wts, V, u[2], &Zw, &eg);
  out->tok_target = t0;
  out->flag_target = eg < 1e-6 ? ORC_FLAG_CDF_EDGE : 0u;
}

/* The whole round for ONE image (Algorithm 1 Steps 2, 4, 5, 6 on given logits).
 *   cond, uncond [H, W, V] (uncond may be NULL), draft_lo [h, w, V],
 *   draft_tok_lo [h, w], nn [V, pool_k] or NULL.
 * Outputs (any may be NULL): out_tok [H,W]; reject, expand [H,W] bytes;
 *   p_tok, q_tok, accept_prob [H,W] double; flags [H,W] (ORC_FLAG_* of the
 *   decision actually used at that position); cand_tok [H,W] = the draw that
 *   position would receive if it lies in R_X; counts[3] = |R_T|, |R_X|, t_0. */
void orc_round_image(const orc_params* P, const void* cond, const void* uncond,
                     const void* draft_lo, const int32_t* draft_tok_lo, const uint16_t* nn,
                     int32_t* out_tok, uint8_t* reject, uint8_t* expand, double* p_tok,
                     double* q_tok, double* accept_prob, uint32_t* flags, int32_t* cand_tok,
                     int32_t* counts) {
  const int H = P->H, W = P->W, V = P->V, r = P->r, h = H / r, w = W / r, N = H * W;
  const size_t esz = P->dtype == ORC_BF16 ? 2 : 4;
  float* zq = (float*)malloc((size_t)V * sizeof(float));
  float* zt = (float*)malloc((size_t)V * sizeof(float));
  double* q = (double*)malloc((size_t)V * sizeof(double));
  double* p = (double*)malloc((size_t)V * sizeof(double));
  double* pp = (double*)malloc((size_t)V * sizeof(double));
  double* wts = (double*)malloc((size_t)V * sizeof(double));
  orc_position* rec = (orc_position*)malloc((size_t)N * sizeof(orc_position));
  uint8_t* rej = (uint8_t*)malloc((size_t)N);
  uint8_t* exp_ = (uint8_t*)malloc((size_t)N);

  /* parent cell by parent cell, so the draft row is turned into q once and
   * shared by its r*r children (q_{ij} = q_{i/r, j/r}) */
  for (int a = 0; a < h; ++a)
    for (int c = 0; c < w; ++c) {
      const size_t cell = (size_t)a * w + c;
      orc_preprocess_row((const char*)draft_lo + cell * V * esz, NULL, P->dtype, V, 0.0f,
                         P->temperature, zq);
      float theta_q = orc_topk_threshold(zq, V, P->top_k);
      double mq, Zq;
      orc_softmax_masked(zq, V, theta_q, q, &mq, &Zq);
      const int tok = draft_tok_lo[cell]; /* x~ of all children */
      for (int di = 0; di < r; ++di)
        for (int dj = 0; dj < r; ++dj) {
          const int i = a * r + di, j = c * r + dj;
          const size_t t = (size_t)i * W + j;
          const char* crow = (const char*)cond + t * V * esz;
          const char* urow = uncond ? (const char*)uncond + t * V * esz : NULL;
          orc_preprocess_row(crow, urow, P->dtype, V, P->cfg_scale, P->temperature, zt);
          visit_position(P, zt, q, tok, nn, (uint32_t)t, p, pp, wts, &rec[t]);
          rej[t] = rec[t].accepted ? 0 : 1;
        }
    }

  int t0 = orc_expand(rej, H, W, P->radius, P->clip_before_first, exp_);
  int n_rej = 0, n_exp = 0;
  for (int t = 0; t < N; ++t) {
    n_rej += rej[t];
    n_exp += exp_[t];
    const int tok = draft_tok_lo[(size_t)(t / W / r) * w + (size_t)(t % W / r)];
    /* which draw applies at t if t is in R_X */
    int use_residual;
    if (P->resample_mode == ORC_RESAMPLE_RESIDUAL_ALL) use_residual = 1;
    else if (P->resample_mode == ORC_RESAMPLE_TARGET_ALL) use_residual = 0;
    else if (P->resample_mode == ORC_RESAMPLE_ISOLATED_RESIDUAL) {
      /* rejected, and t would NOT have been swept in had it been accepted: no
       * other rejected position has t inside its N(.,l) -- where the t_0 of
       * Eq. 6 is then the first rejection among the others, so the first
       * rejected position of the image is never covered when clipping is on */
      use_residual = rej[t];
      for (int v = 0; v < N && use_residual; ++v)
        if (v != t && rej[v] && abs(v / W - t / W) <= P->radius && abs(v % W - t % W) <= P->radius &&
            (!P->clip_before_first || t != t0))
          use_residual = 0;
    } else use_residual = rej[t];
    int cand = use_residual ? rec[t].tok_residual : rec[t].tok_target;
    uint32_t f = rec[t].flags | (use_residual ? rec[t].flag_residual : rec[t].flag_target);
    if (out_tok) out_tok[t] = exp_[t] ? cand : tok;
    if (cand_tok) cand_tok[t] = cand;
    if (reject) reject[t] = rej[t];
    if (expand) expand[t] = exp_[t];
    if (p_tok) p_tok[t] = rec[t].p_tok;
    if (q_tok) q_tok[t] = rec[t].q_tok;
    if (accept_prob) accept_prob[t] = rec[t].accept_prob;
    if (flags) flags[t] = f;
  }
  if (counts) {
    counts[0] = n_rej;
    counts[1] = n_exp;
    counts[2] = t0;
  }
  free(zq); free(zt); free(q); free(p); free(pp); free(wts); free(rec); free(rej); free(exp_);
}

/* ------------------------------------------- small helpers used by the pins */

/* q, p and p' rows for one position, exposed so tests can check invariants.
 * cond/uncond/draft point at the rows themselves. */
void orc_position_distributions(const orc_params* P, const void* cond_row, const void* uncond_row,
                                const void* draft_row, int tok, const uint16_t* nn, double* q,
                                double* p, double* p_prime, double* pooled_mass) {
  const int V = P->V;
  float* z = (float*)malloc((size_t)V * sizeof(float));
  double m, Z, gap;
  int J;
  orc_preprocess_row(draft_row, NULL, P->dtype, V, 0.0f, P->temperature, z);
  orc_softmax_masked(z, V, orc_topk_threshold(z, V, P->top_k), q, &m, &Z);
  orc_preprocess_row(cond_row, uncond_row, P->dtype, V, P->cfg_scale, P->temperature, z);
  orc_softmax_masked(z, V, orc_topk_threshold(z, V, P->top_k), p, &m, &Z);
  const uint16_t* nn_row = (P->pool_k > 1 && nn) ? nn + (size_t)tok * P->pool_k : NULL;
  *pooled_mass = orc_pool(p, V, nn_row, P->pool_k, (double)P->pool_delta, tok, p_prime, &J, &gap);
  free(z);
}

/* Histogram of inverse-CDF outcomes over the full 24-bit grid of uniforms
 * u = n * 2^-24, n in [n_begin, n_end): used by the exhaustive exactness pin. */
void orc_inverse_cdf_histogram(const double* w, int V, uint32_t n_begin, uint32_t n_end,
                               int64_t* hist) {
  for (uint32_t n = n_begin; n < n_end; ++n) {
    int tok = orc_inverse_cdf(w, V, (double)n * (1.0 / 16777216.0), NULL, NULL);
    if (tok >= 0) hist[tok] += 1;
  }
}

/* Step 1 on given logits: one token per low-res cell from q (after temperature /
 * top-k) by inverse CDF in ascending token id, uniform = word 0 of the tag-1
 * Philox stream at (cell, image, round).  edge[cell] (may be NULL) = 1 where the
 * uniform lies within 1e-6 of an edge of the chosen CDF bin. */
void orc_sample_draft_tokens(const orc_params* P, const void* draft_lo, int32_t* draft_tok_lo,
                             uint8_t* edge) {
  const int V = P->V, h = P->H / P->r, w = P->W / P->r;
  const size_t esz = P->dtype == ORC_BF16 ? 2 : 4;
  float* z = (float*)malloc((size_t)V * sizeof(float));
  double* q = (double*)malloc((size_t)V * sizeof(double));
  for (int cell = 0; cell < h * w; ++cell) {
    double m, Z, u[3], gap;
    orc_preprocess_row((const char*)draft_lo + (size_t)cell * V * esz, NULL, P->dtype, V, 0.0f,
                       P->temperature, z);
    orc_softmax_masked(z, V, orc_topk_threshold(z, V, P->top_k), q, &m, &Z);
    orc_position_uniforms(P->seed, P->image, (uint32_t)cell, P->round, 1u, u);
    draft_tok_lo[cell] = orc_inverse_cdf(q, V, u[0], NULL, &gap);
    if (edge) edge[cell] = gap < 1e-6;
  }
  free(z);
  free(q);
}

/* The redraw of R_X executed step by step (Sec. 3.4, Algorithm 1 Step 6).  The target model
 * is called once per sequential step s = 1 .. n_steps of the schedule; a call yields logits for
 * the whole grid given the tokens decoded so far, and the positions with step(t) == s take their
 * token from them: one draw from the target distribution (CFG, temperature, top-k as in the round)
 * by inverse CDF in ascending token id.  Here the model calls are an input: cond_steps[s - 1]
 * (and uncond_steps[s - 1], or uncond_steps == NULL) is the [H*W, V] logit tensor of call s.
 * Reading: the uniform of position t at step s is word 0 of the Philox stream with counter
 * (t, image, round, 1 + s) -- tag 0 holds the round's own uniforms and tag 1 the drafter's draw,
 * so the redraw's numbers are new ones and a position redrawn in two different rounds or steps
 * never reuses a uniform (the paper does not say how the redraw is seeded).
 *   step [H*W]  the schedule (0 outside R_X);   tok [H*W] in/out: positions outside R_X keep
 *   their token;   edge [H*W] out, may be NULL: 1 where the uniform lies within 1e-6 of an edge
 *   of the chosen CDF bin.
 * Returns the number of target-model calls made (the NFE of the redraw): n_steps. */
int orc_redraw_loop(const orc_params* P, const int32_t* step, int n_steps, const void* const* cond_steps,
                    const void* const* uncond_steps, int32_t* tok, uint8_t* edge) {
  const int V = P->V, N = P->H * P->W;
  const size_t esz = P->dtype == ORC_BF16 ? 2 : 4;
  float* z = (float*)malloc((size_t)V * sizeof(float));
  double* p = (double*)malloc((size_t)V * sizeof(double));
  int calls = 0;
  if (edge) memset(edge, 0, (size_t)N);
  for (int s = 1; s <= n_steps; ++s) {
    const char* cond = (const char*)cond_steps[s - 1];
    const char* uncond = uncond_steps ? (const char*)uncond_steps[s - 1] : NULL;
    ++calls;
    for (int t = 0; t < N; ++t) {
      if (step[t] != s) continue;
      double m, Z, u[3], gap;
      orc_preprocess_row(cond + (size_t)t * V * esz, uncond ? uncond + (size_t)t * V * esz : NULL, P->dtype, V,
                         P->cfg_scale, P->temperature, z);
      orc_softmax_masked(z, V, orc_topk_threshold(z, V, P->top_k), p, &m, &Z);
      orc_position_uniforms(P->seed, P->image, (uint32_t)t, P->round, 1u + (uint32_t)s, u);
      tok[t] = orc_inverse_cdf(p, V, u[0], NULL, &gap);
      if (edge) edge[t] = gap < 1e-6;
    }
  }
  free(z);
  free(p);
  return calls;
}

/* Step 7 stand-in.  The paper's D_r is a trained network; the stand-in keeps the
 * one property the round relies on, D_r(U_r(y)) = y for the replicating U_r:
 * y[a][c] is the token that occurs most often among the r x r tokens
 * x[a r + di][c r + dj]; among tokens with the same count, the one that occurs
 * first in raster order of the block. */
void orc_downsample_majority(const int32_t* x, int H, int W, int r, int32_t* y) {
  const int h = H / r, w = W / r;
  for (int a = 0; a < h; ++a)
    for (int c = 0; c < w; ++c) {
      int best_tok = -1, best_count = 0;
      for (int s = 0; s < r * r; ++s) {
        const int tok = x[(a * r + s / r) * W + c * r + s % r];
        int count = 0;
        for (int s2 = 0; s2 < r * r; ++s2)
          if (x[(a * r + s2 / r) * W + c * r + s2 % r] == tok) ++count;
        if (count > best_count) { /* strict: an earlier token keeps a tie */
          best_count = count;
          best_tok = tok;
        }
      }
      y[a * w + c] = best_tok;
    }
}
