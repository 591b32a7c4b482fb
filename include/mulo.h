/*
 * mulo.h -- C ABI of the B200 (sm_100a) draft-and-verify round of Multi-Scale
 * Local Speculative Decoding (MuLo-SD) for autoregressive image generation.
 *
 * One speculative round over an H x W grid of image tokens, for B independent
 * images, given the target model's logits at every position and the drafter's
 * logits on the (H/r) x (W/r) low-resolution grid:
 *
 *   up-sample draft tokens and draft distributions to the target grid
 *   -> target / draft probabilities over the vocabulary (CFG, temperature, top-k)
 *   -> acceptance test  u < min(1, P / q(x~))        (Sec. 3.1, Eq. 1 and Eq. 3)
 *   -> rejection mask R_T, first rejection t_0       (Sec. 3.3)
 *   -> local expansion R_X                           (Sec. 3.3, Eq. 6-7)
 *   -> parallel inverse-CDF redraw of R_X            (Eq. 2; Algorithm 1 Step 6)
 * and, for the scheduler of the redraw, the rejection islands of R_X (Sec. 3.4, Eq. 8).
 *
 * Conventions for every call
 *   - All tensor arguments are DEVICE pointers to caller-owned, contiguous,
 *     row-major memory, 16-byte aligned, unless the name says "host".  The
 *     library never allocates or frees device memory; scratch space is the
 *     workspace the caller hands to mulo_set_workspace.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls validate their arguments on the host, enqueue kernels on the stream
 *     and return; outputs are defined once the stream has been synchronised.  Nothing a
 *     call does blocks or leaves the stream, so calls can be captured into a CUDA graph
 *     (parameters, `round` included, are frozen at capture) unless their text says otherwise.
 *   - A context is bound to one device.  Kernels are launched on the calling thread's
 *     CURRENT device, so that device must be the context's: a call made while another
 *     device is current returns MULO_ERR_INVALID_ARG before anything is enqueued.
 *   - Errors are return codes.  An invalid argument is detected before anything
 *     is launched.  Kernels never trap; contract violations they can see (a
 *     draft token with zero draft probability, a token id outside [0, V)) set a
 *     bit that mulo_poll_device_status reports.
 *   - Positions are raster indices t = i * W + j.  Bit masks hold one bit per
 *     position: bit (j % 32) of word (b * H + i) * ceil(W / 32) + j / 32.
 *   - Logit tensors share one dtype (fp32, or bf16 as raw 16-bit patterns) and
 *     must be finite.  V must be a multiple of 8 and at most 65536.
 *   - Uniform random numbers: Philox4x32-10 with key (seed low word, seed high
 *     word) and counter (position t, image b + image_offset, round, 0); output
 *     word 0 drives the acceptance test, word 1 the residual draw, word 2 the
 *     draw from the target distribution; u = (word >> 8) * 2^-24.
 */
#ifndef MULO_H_
#define MULO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mulo_ctx mulo_ctx; /* opaque; one per device and host thread */

typedef enum {
  MULO_OK = 0,
  MULO_ERR_INVALID_ARG = 1, /* NULL / misaligned pointer, bad shape or parameter        */
  MULO_ERR_UNSUPPORTED = 2, /* valid but outside what the kernels handle (see limits)   */
  MULO_ERR_WORKSPACE = 3,   /* no workspace set, or too small for these parameters      */
  MULO_ERR_CUDA = 4,        /* a CUDA runtime call failed (also: no usable device)      */
  MULO_ERR_TIMEOUT = 5      /* a bounded device-side wait gave up (MULO_DEV_TIMEOUT): the
                               results of the calls since the last poll are invalid     */
} mulo_status;

typedef enum { MULO_F32 = 0, MULO_BF16 = 1 } mulo_dtype;

typedef enum {
  MULO_ACCEPT_RATIO = 0,    /* Eq. 1 with Eq. 3's pooled numerator: u < min(1, P/q(x~))  */
  MULO_ACCEPT_THRESHOLD = 1 /* Eq. 5: accept iff pooled target mass P >= tau (no q, no u) */
} mulo_accept_mode;

typedef enum {
  MULO_RESAMPLE_MIXED = 0,        /* rejected positions: residual of Eq. 2; the rest of R_X:
                                     the target distribution (Algorithm 1 Step 6)            */
  MULO_RESAMPLE_RESIDUAL_ALL = 1, /* every position of R_X from the residual                  */
  MULO_RESAMPLE_TARGET_ALL = 2,   /* every position of R_X from the target distribution       */
  MULO_RESAMPLE_ISOLATED_RESIDUAL = 3 /* residual only for a rejected position that no other
                                     rejection would have swept in; target distribution for
                                     the rest of R_X (exact for independent draft tokens)   */
} mulo_resample_mode;

/* device status bits (mulo_poll_device_status) */
#define MULO_DEV_ZERO_DRAFT_PROB 1u /* some draft token had q(x~) == 0                    */
#define MULO_DEV_BAD_TOKEN 2u       /* some token / neighbour id was outside [0, V)        */
#define MULO_DEV_DENSE_FALLBACK 4u  /* informational: a row left the fast top-k path       */
#define MULO_DEV_TIMEOUT 8u         /* a bounded device-side wait gave up: results invalid */

typedef struct mulo_params {
  int32_t B, H, W;       /* images, target grid; the draft grid is (H/r) x (W/r)            */
  int32_t V;             /* vocabulary size: multiple of 8, <= 65536                         */
  int32_t r;             /* resolution ratio s_p / s_q >= 1; H % r == 0 and W % r == 0       */
  int32_t logit_dtype;   /* mulo_dtype of all three logit tensors                            */
  float temperature;     /* > 0; logits are multiplied by fp32(1 / temperature)              */
  int32_t top_k;         /* <= 0 or >= V: off.  Otherwise keep every entry >= the k-th
                            largest value of the row (ties kept); same k for target/draft   */
  float cfg_scale;       /* s of l = l_u + s (l_c - l_u); used iff an unconditional tensor
                            is passed                                                        */
  int32_t accept_mode;   /* mulo_accept_mode                                                 */
  float tau;             /* Eq. 5 threshold (MULO_ACCEPT_THRESHOLD only)                     */
  int32_t pool_k;        /* codebook neighbourhood size k of Eq. 3; <= 1 turns pooling off;
                            at most 2048                                                     */
  float pool_delta;      /* delta of Eq. 4: the pooled neighbours may add < delta of mass    */
  int32_t radius;        /* l of Eq. 6, 0 <= l <= 31; l rounds of 3x3 growth                 */
  int32_t clip_before_first; /* non-zero: keep Eq. 6's clause u >= t_0                       */
  int32_t resample_mode; /* mulo_resample_mode                                               */
  uint64_t seed;         /* Philox key                                                       */
  uint32_t round;        /* speculative round index (Philox counter word 2)                  */
  uint32_t image_offset; /* added to the image index b in Philox counter word 1, so that a
                            batch split over several calls or devices draws the same numbers */
} mulo_params;

/* ---- context, workspace, diagnostics (no counterpart in the paper) ------------------- */

/* Creates a context bound to CUDA device `device` (queries its limits, raises the
 * kernels' dynamic shared-memory caps).  Returns MULO_ERR_CUDA if the device cannot be
 * used.  The context is host memory owned by the library until mulo_destroy. */
mulo_status mulo_create(mulo_ctx** out, int device);
void mulo_destroy(mulo_ctx* ctx);
const char* mulo_status_string(mulo_status s);

/* Bytes of device scratch that calls with these parameters need (status word, per-position
 * accept flags and candidate tokens, the list of positions the fast kernel leaves to the
 * general routines): 13 bytes per grid position plus padding. */
mulo_status mulo_workspace_bytes(const mulo_params* p, size_t* bytes);
/* Hands the library a caller-owned device buffer (256-byte aligned).  It must stay valid
 * and must not be shared by calls that overlap on the device.  The first 256 bytes hold
 * the device status word; this call clears it (on the default stream, synchronously). */
mulo_status mulo_set_workspace(mulo_ctx* ctx, void* dev_ptr, size_t bytes);
/* Synchronises `stream`, reads and clears the device status bits (MULO_DEV_*).  *flags is
 * written in every case that got as far as reading them; the return value is
 * mulo_status_of_device_flags(*flags): MULO_ERR_TIMEOUT if a kernel's bounded wait on one of
 * its own copies gave up.  A CTA whose wait gave up writes nothing further (its remaining
 * rows keep whatever the workspace held), waits a bounded time for its copies in flight and
 * returns; the other CTAs finish.  The context stays usable. */
mulo_status mulo_poll_device_status(mulo_ctx* ctx, void* stream, uint32_t* flags);
/* The status that a set of device status bits maps to (host arithmetic only): MULO_ERR_TIMEOUT
 * if MULO_DEV_TIMEOUT is among them, else MULO_OK -- the other bits are reports, not errors. */
mulo_status mulo_status_of_device_flags(uint32_t flags);
/* Synchronises `stream`, reads and clears five counters kept next to the status bits:
 * counts[0] rows that mulo_round's fast kernel handed to the general routines, and of those
 * counts[1] because a candidate list was full, counts[2] because fewer than top_k candidates
 * passed the predicted pivot, counts[3] because the k-th largest lay above the selection
 * histogram, counts[4] because too many entries tied near it (the target rows under a draft
 * row that was handed over follow it without a reason of their own).  Results are the same
 * either way; a large counts[0] means the rows are far from what the predictor expects and
 * the round runs at the general kernel's speed. */
mulo_status mulo_poll_fallback_counts(mulo_ctx* ctx, void* stream, uint32_t counts[5]);
/* Number of kernels this context has launched so far. */
mulo_status mulo_kernel_launches(const mulo_ctx* ctx, uint64_t* count);
/* mulo_round picks between four row kernels, mulo_sample_draft between the last two.  All
 * compute the same function; a row a fast kernel cannot handle is redone by the general routines.
 *   MULO_KERNEL_FULL     top-k off (the paper's default sampling), V a multiple of 2048 (bf16) or
 *                        1024 (fp32), the rows of one position within a CTA's shared memory (e.g.
 *                        V <= 16384 in bf16 with classifier-free guidance): rows are made resident
 *                        in shared memory and every entry is exponentiated once; with Eq. 5 and
 *                        redraws from the target distribution the draft logits are not read;
 *   MULO_KERNEL_LANE     top-k on, pooling off, V a multiple of 4096 (bf16) or 2048 (fp32) and
 *                        at most 16384: every thread of a CTA owns a contiguous range of the
 *                        vocabulary, rows are streamed once through per-warp shared-memory rings;
 *   MULO_KERNEL_STREAM   top-k on, V >= 1024 (with pooling, V <= 16384), any other shape: rows
 *                        streamed once in chunks, candidates compacted per segment;
 *   MULO_KERNEL_GENERAL  everything else (top-k off, tiny vocabularies): one CTA per row, the
 *                        row read several times (from L2 after the first).
 * mulo_round_kernel reports the choice for these parameters (and with or without an unconditional
 * tensor) on this context (host arithmetic only; nothing is launched).  mulo_set_general_path_only(on != 0) makes the context always use
 * the general kernel (for testing and comparison). */
typedef enum {
  MULO_KERNEL_GENERAL = 0, MULO_KERNEL_STREAM = 1, MULO_KERNEL_LANE = 2, MULO_KERNEL_FULL = 3
} mulo_kernel;
mulo_status mulo_round_kernel(const mulo_ctx* ctx, const mulo_params* p, int has_uncond, int* kernel);
mulo_status mulo_set_general_path_only(mulo_ctx* ctx, int on);
/* Optional device timing of the fused row kernel (the launch that reads the logits):
 * mulo_set_timing prepares CUDA event pairs for up to max_launches (<= 4096) calls of
 * mulo_round (0 turns timing off); every mulo_round then records an event on its stream
 * before and after that kernel.  mulo_read_timing waits for the recorded launches, returns
 * their summed duration in milliseconds and their number, and starts a new series. */
mulo_status mulo_set_timing(mulo_ctx* ctx, int max_launches);
mulo_status mulo_read_timing(mulo_ctx* ctx, double* row_kernel_ms, uint64_t* row_kernel_launches);

/* ---- the four stages ------------------------------------------------------------------ */

/* Step 2 of the pipeline (Sec. 3.2: x~ = U_r(y~), r^2 times as many tokens) with the
 * nearest-neighbour stand-in for U_r, plus the part of the pooled acceptance rule (Eq. 3)
 * that needs only the drafter: per low-res cell the draft row's top-k threshold theta_q,
 * maximum m_q and partition sum Z_q (so that q(x) = [z >= theta_q] exp(z - m_q) / Z_q),
 * and q(x~) at every target position.
 *   draft_logits_lo [B, h, w, V]   in
 *   draft_tok_lo    [B, h, w]      in   int32 token ids
 *   nn              [V, pool_k]    in   uint16; unused here, may be NULL
 *   draft_tok_hi    [B, H, W]      out  x~[b,i,j] = y~[b,i/r,j/r]
 *   draft_stats_lo  [B, h, w, 4]   out  fp32 (theta_q, m_q, Z_q high part, Z_q low part):
 *                                       Z_q = hi + lo; theta_q = -inf if top-k is off
 *   q_tok_hi        [B, H, W]      out  fp32 q(x~)                                        */
mulo_status mulo_upsample_pool(mulo_ctx* ctx, const mulo_params* p, const void* draft_logits_lo,
                               const int32_t* draft_tok_lo, const uint16_t* nn,
                               int32_t* draft_tok_hi, float* draft_stats_lo, float* q_tok_hi,
                               void* stream);

/* Steps 3-4: target probabilities (CFG mix l_u + s (l_c - l_u), temperature, top-k, softmax;
 * Supp. "Sampling"), pooled mass P over A_{k,delta}(x~) (Eq. 3-4; Algorithm 1), and the
 * acceptance decision (Eq. 1, or Eq. 5 in threshold mode).
 *   tgt_cond, tgt_uncond [B, H, W, V]  in   (tgt_uncond may be NULL: no CFG)
 *   draft_logits_lo, draft_stats_lo, draft_tok_hi, nn   in   as above (nn required iff pool_k > 1;
 *                                      nn[x][0] must be x, the rest distinct and != x)
 *   p_tok, q_tok, accept_prob [B, H, W] out  fp32 p(x~), q(x~), min(1, P/q(x~)) (or P in threshold mode)
 *   reject_bits  [B, H, ceil(W/32)]    out  uint32, 1 = rejected (R_T)
 *   n_reject     [B]                   out  |R_T|
 *   first_reject [B]                   out  t_0, or H*W if nothing was rejected
 * Needs the workspace. */
mulo_status mulo_verify(mulo_ctx* ctx, const mulo_params* p, const void* tgt_cond,
                        const void* tgt_uncond, const void* draft_logits_lo,
                        const float* draft_stats_lo, const int32_t* draft_tok_hi,
                        const uint16_t* nn, float* p_tok, float* q_tok, float* accept_prob,
                        uint32_t* reject_bits, int32_t* n_reject, int32_t* first_reject,
                        void* stream);

/* Step 5: R_X = union over rejected t of N(t, l), N(t, l) = {u : |i_u - i_t| <= l,
 * |j_u - j_t| <= l, u >= t_0} (Eq. 6-7).
 *   reject_bits, first_reject   in
 *   expand_bits [B, H, ceil(W/32)]  out   n_expand [B]  out  |R_X|                        */
mulo_status mulo_local_reject_expand(mulo_ctx* ctx, const mulo_params* p,
                                     const uint32_t* reject_bits, const int32_t* first_reject,
                                     uint32_t* expand_bits, int32_t* n_expand, void* stream);

/* Schedule of the redraw (Sec. 3.4): different islands are redrawn concurrently; within an
 * island the target model advances row by row, left to right, with a ZipAR-style row window:
 * a position may be decoded one step after the island's previous position in its row, and one
 * step after the island's positions of the row above up to `window - 1` columns beyond it,
 *   step(t) = 1 + max(step of the island's earlier positions in row i,
 *                     step of the island's positions (i - 1, j') with j' <= j + window - 1).
 * The paper names the strategy and the window (16); this recurrence is the reading taken.
 * A full H x W island takes W + (H - 1) window steps instead of H W.  H * W <= 16384.
 *   labels  [B, H, W]  in   island numbers from mulo_islands (0 outside R_X)
 *   window             >= 1
 *   step    [B, H, W]  out  1-based sequential target-model step of the position, 0 outside R_X
 *   n_steps [B]        out  sequential steps the image needs (the largest step)               */
mulo_status mulo_island_schedule(mulo_ctx* ctx, const mulo_params* p, const int32_t* labels,
                                 int32_t window, int32_t* step, int32_t* n_steps, void* stream);

/* Step 1 on given logits (Sec. 3.2): the drafter's own draw y~ ~ q, one token per low-res cell,
 * by inverse CDF in ascending token id over q = softmax(topk(l_q / T)) (same temperature and
 * top-k as the round).  The uniform is word 0 of the Philox stream with counter
 * (cell index a * w + c, image b + image_offset, round, 1): the last counter word tells it
 * apart from the round's own uniforms, which use 0 there.  Needs a workspace (status word).
 *   draft_logits_lo [B, h, w, V]  in      draft_tok_lo [B, h, w]  out                       */
mulo_status mulo_sample_draft(mulo_ctx* ctx, const mulo_params* p, const void* draft_logits_lo,
                              int32_t* draft_tok_lo, void* stream);

/* Step 7 stand-in (Sec. 3.2: y = D_r(x), the prefix of the next low-resolution draft).  The
 * paper's D_r is a trained network; this call keeps the one property the round relies on,
 * D_r(U_r(y)) = y for the replicating up-sampler: tok_lo[a][c] is the token that occurs most
 * often in the r x r block tok_hi[a r .. a r + r - 1][c r .. c r + r - 1]; among tokens with
 * the same count, the one that comes first in raster order of the block.  r <= 16.
 *   tok_hi [B, H, W]  in      tok_lo [B, h, w]  out                                          */
mulo_status mulo_downsample(mulo_ctx* ctx, const mulo_params* p, const int32_t* tok_hi,
                            int32_t* tok_lo, void* stream);

/* Rejection islands (Sec. 3.4, Eq. 8): {I_m} = CC_8(R_X), the 8-connected components of R_X
 * on the token grid (two positions are neighbours when both coordinates differ by at most
 * one), which a scheduler redraws concurrently.  Uses B, H, W of `p`; H * W <= 16384, else
 * MULO_ERR_UNSUPPORTED.  Needs no workspace.
 *   expand_bits [B, H, ceil(W/32)]   in   R_X
 *   labels      [B, H, W]            out  0 outside R_X, else the island's number m in 1..M.
 *                                         Islands are numbered by the raster index of their
 *                                         first position (the paper leaves the order open).
 *   n_islands   [B]                  out  M
 *   max_islands                           rows of the two tables below per image (>= 0)
 *   island_rows [B, max_islands, 2]  out, may be NULL: first and last grid row of island m at
 *                                         entry m - 1; entries from M on are (-1, -1)
 *   island_size [B, max_islands]     out, may be NULL: number of positions; 0 from M on
 * With M > max_islands the labels and n_islands are still complete; the tables hold the
 * first max_islands islands. */
mulo_status mulo_islands(mulo_ctx* ctx, const mulo_params* p, const uint32_t* expand_bits,
                         int32_t* labels, int32_t* n_islands, int32_t max_islands,
                         int32_t* island_rows, int32_t* island_size, void* stream);

/* Step 6 on given logits: every position of R_X is redrawn in parallel by inverse CDF over
 * w(x) = max(0, p'(x) - lambda q(x)) in ascending token id, lambda = 1 (Eq. 2) or 0
 * (Algorithm 1 Step 6) as resample_mode says; p' is p with the pooled mass moved onto x~.
 * A residual without mass falls back to lambda = 0.  Positions outside R_X keep x~.
 *   out_tok [B, H, W]  out  int32                                                         */
mulo_status mulo_resample(mulo_ctx* ctx, const mulo_params* p, const void* tgt_cond,
                          const void* tgt_uncond, const void* draft_logits_lo,
                          const float* draft_stats_lo, const int32_t* draft_tok_hi,
                          const uint16_t* nn, const uint32_t* reject_bits,
                          const uint32_t* expand_bits, int32_t* out_tok, void* stream);

/* ---- the redraw of R_X, step by step (Sec. 3.4, Algorithm 1 Step 6) ------------------------ */

/* Sorts the positions of R_X by their step of the schedule (mulo_island_schedule), on the device:
 *   step         [B, H, W]             in   1-based step of each position, 0 outside R_X
 *   max_step                                an upper bound of the steps present, 1 <= max_step <= H W
 *                                           (positions with a larger step are left out)
 *   pos_list     [B H W]               out  position indices b H W + t, the positions of step 1 first,
 *                                           then step 2, ...; order within a step unspecified
 *   step_offsets [2 (max_step + 2)]    out  entry s (1 <= s <= max_step) = where step s starts in
 *                                           pos_list, entry max_step + 1 = where the last step ends;
 *                                           the second half of the array is scratch
 * Three small launches, no host round-trip.  Needs no workspace. */
mulo_status mulo_redraw_plan(mulo_ctx* ctx, const mulo_params* p, const int32_t* step, int32_t max_step,
                             int32_t* pos_list, int32_t* step_offsets, void* stream);
/* One sequential step s of the redraw: every position of step s takes a new token, drawn from the
 * target distribution p(. | the given logits) -- CFG mix, temperature and top-k as in the round,
 * inverse CDF in ascending token id.  The logits stand for the target model's call number s (the
 * model is not part of this library): tgt_cond / tgt_uncond are [B, H, W, V] tensors of which only
 * the rows of this step's positions are read.  The uniform of position t is word 0 of Philox4x32-10
 * at counter (t, image_offset + b, round, 1 + s): a stream of its own beside the round's (tag 0) and
 * the drafter's (tag 1); the paper does not say how the redraw is seeded.  One launch whose grid
 * does not depend on how many positions the step has (their number stays on the device).
 *   s, max_step                     1 <= s <= max_step, max_step as given to mulo_redraw_plan
 *   pos_list, step_offsets     in   from mulo_redraw_plan
 *   out_tok [B, H, W]          in/out  int32; only this step's positions are written           */
mulo_status mulo_redraw_step(mulo_ctx* ctx, const mulo_params* p, int32_t s, int32_t max_step,
                             const int32_t* pos_list, const int32_t* step_offsets, const void* tgt_cond,
                             const void* tgt_uncond, int32_t* out_tok, void* stream);

/* ---- the fused round ------------------------------------------------------------------- */

/* The four stages in one pass: every logit row is read from HBM once.  Results are those
 * of mulo_upsample_pool -> mulo_verify -> mulo_local_reject_expand -> mulo_resample, with one
 * exception: with MULO_ACCEPT_THRESHOLD and MULO_RESAMPLE_TARGET_ALL (Eq. 5 as printed, every
 * redraw from the target distribution) neither the decision nor any draw depends on the draft
 * distribution, so q_tok, if given, is filled with zeros, and where the resident-row kernel
 * runs (MULO_KERNEL_FULL) draft_logits_lo is not read at all (it must still be a valid pointer).
 *   p_tok, q_tok, accept_prob may be NULL (skipped).  Needs the workspace. */
mulo_status mulo_round(mulo_ctx* ctx, const mulo_params* p, const void* tgt_cond,
                       const void* tgt_uncond, const void* draft_logits_lo,
                       const int32_t* draft_tok_lo, const uint16_t* nn, int32_t* out_tok,
                       uint32_t* reject_bits, uint32_t* expand_bits, float* p_tok, float* q_tok,
                       float* accept_prob, int32_t* n_reject, int32_t* n_expand,
                       int32_t* first_reject, void* stream);

/* mulo_round for callers whose tensors live in HOST memory (pinned memory copies fastest):
 * copies the inputs into `arena` (caller-owned device memory of at least
 * mulo_round_host_arena_bytes, 256-byte aligned; it also serves as the workspace, replacing
 * any set before), runs the round, copies the results back and synchronises `stream`
 * before returning.  All tensor arguments are HOST pointers; optional ones may be NULL. */
mulo_status mulo_round_host_arena_bytes(const mulo_params* p, int has_uncond, size_t* bytes);
mulo_status mulo_round_host(mulo_ctx* ctx, const mulo_params* p, void* arena, size_t arena_bytes,
                            const void* tgt_cond, const void* tgt_uncond,
                            const void* draft_logits_lo, const int32_t* draft_tok_lo,
                            const uint16_t* nn, int32_t* out_tok, uint32_t* reject_bits,
                            uint32_t* expand_bits, float* p_tok, float* q_tok,
                            float* accept_prob, int32_t* n_reject, int32_t* n_expand,
                            int32_t* first_reject, void* stream);

/* ---- a round for callers that cannot allocate device memory ---------------------------- */

/* The paper has no counterpart to this call; it exists for deployment reasons only.
 *
 * mulo_round needs a scratch buffer (one accept flag and two candidate tokens per grid
 * position, plus the device status word) that somebody has to allocate.  Some hosts
 * cannot: an inference server whose memory pool has already claimed every free byte of
 * HBM, so that a cudaMalloc at request time fails; a plug-in that runs inside such a
 * server and is handed its inputs and outputs but no allocator; a latency-critical loop
 * in which the implicit device synchronisation of cudaMalloc / cudaFree is not acceptable.
 * mulo_round_static is mulo_round for them.  Its scratch is a fixed array of
 * MULO_STATIC_SCRATCH_BYTES that is part of the library image: every GPU on which the
 * library runs a kernel holds that much memory from then until the process exits, whether
 * or not this call is ever used.  Nothing in this call allocates or frees memory, on the
 * device or through any library that might.
 *
 *   - Same inputs, outputs and results as mulo_round (the same kernels run).  The
 *     workspace handed to mulo_set_workspace, if any, is neither needed nor touched.
 *   - Size limit: mulo_workspace_bytes(p) must not exceed MULO_STATIC_SCRATCH_BYTES
 *     (about 80,000 grid positions per call, e.g. 19 images of 64 x 64).  A larger
 *     request returns MULO_ERR_WORKSPACE before anything is launched; split the batch
 *     over several calls (image_offset keeps the random streams aligned).  Every other
 *     refusal (a NULL or misaligned tensor, bad parameters, another device current)
 *     also comes before the array is touched.
 *   - device_status [1], DEVICE pointer, may be NULL: receives the MULO_DEV_* bits this
 *     call raised (the call clears the bits first, so they describe this call alone).
 *   - The first call on a device looks up the array's device address (once per device, with
 *     that device made current for the lookup).  Make that first call outside any stream
 *     capture.
 *   - There is one array per device and every call uses it.  It keeps whatever the last
 *     call left there; the call re-initialises the part that must start at zero and
 *     overwrites the rest before reading it.  Two calls that may run on the same device
 *     at the same time (different streams, different host threads, different contexts)
 *     race on it and give undefined results: order them on one stream or with events. */
#define MULO_STATIC_SCRATCH_BYTES (1u << 20)
mulo_status mulo_round_static(mulo_ctx* ctx, const mulo_params* p, const void* tgt_cond,
                              const void* tgt_uncond, const void* draft_logits_lo,
                              const int32_t* draft_tok_lo, const uint16_t* nn, int32_t* out_tok,
                              uint32_t* reject_bits, uint32_t* expand_bits, float* p_tok,
                              float* q_tok, float* accept_prob, int32_t* n_reject,
                              int32_t* n_expand, int32_t* first_reject, uint32_t* device_status,
                              void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MULO_H_ */
