/*
 * attnfuse: the fused attention kernel of a composed variant
 *     softmax(mask(alibi(rope(Q, K)))) @ V          (paper: Introduction, Sections 3.1 and 4.1)
 * and its backward pass (Section 4.4), hand-written for sm_100a.
 *
 * Conventions for every entry point
 *  - C linkage, plain pointers and sizes.  Unless a parameter says HOST, data pointers are DEVICE
 *    pointers owned by the caller; the library allocates no device memory.
 *  - Tensors are [B, H, S, D] with D contiguous, bf16 (2 bytes per element).  Query-side tensors
 *    have Hq heads, key/value-side tensors Hkv heads; query head h reads kv head h / gqa_group.
 *  - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = default stream)
 *    and the call returns without synchronising.  Outputs are valid once the stream is.
 *  - Argument errors are detected before anything is launched, leave outputs untouched and are
 *    reported by return code; nothing throws or aborts.
 *  - Device-side waits are bounded.  A wait that runs out makes the kernel return early and
 *    records a code that attnfuse_device_status() reports; outputs of that launch are undefined.
 *  - Forward and backward are run-to-run deterministic (no atomics in the data path).
 */
#ifndef ATTNFUSE_H_
#define ATTNFUSE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    AF_OK = 0,
    AF_ERR_NULL = 1,            /* a required pointer is NULL */
    AF_ERR_SHAPE = 2,           /* unsupported or inconsistent sizes (D not 64/128, Hq != Hkv*group, ...) */
    AF_ERR_DTYPE = 3,           /* unsupported element type */
    AF_ERR_ALIGN = 4,           /* pointer not 16-byte aligned or stride not a multiple of 8 elements */
    AF_ERR_SPEC = 5,            /* bad RoPE / mask specification */
    AF_ERR_WORKSPACE = 6,       /* workspace missing or too small */
    AF_ERR_ARCH = 7,            /* current device is not compute capability 10.x */
    AF_ERR_CUDA = 8,            /* a CUDA runtime / driver call failed */
    AF_ERR_DEVICE_TIMEOUT = 9,  /* a bounded device-side wait ran out in an earlier launch */
    AF_ERR_STATIC_LIMIT = 10    /* attnfuse_bwd_static: B*Hq*S exceeds AF_BWD_STATIC_MAX_ROWS */
} af_status;

typedef enum { AF_BF16 = 0, AF_F32 = 1 } af_dtype;

/* Problem geometry.  S is both the query and the key length. */
typedef struct { int B, Hq, Hkv, S, D; } af_shape;

/* Element strides of an input tensor; the D stride is 1.  NULL where accepted = contiguous. */
typedef struct { int64_t b, h, s; } af_strides;

/* RoPE (Section 4.1): NeoX half-swap pairing (i, i + rotary_dim/2), frequency theta^(-2i/rotary_dim),
 * row s of Q and of K sits at position pos_offset + s.  rotary_dim = 0 disables the rotation;
 * otherwise it must be a multiple of 16 and <= D.  Dims >= rotary_dim pass through. */
typedef struct { float theta; int rotary_dim; int pos_offset; } af_rope;

/* Post-matmul score modifiers (Section 3.1: causal, sliding_window, alibi).
 * causal != 0: keep j <= i.  window >= 0: keep |i - j| <= window (with causal: 0 <= i-j <= window);
 * window < 0: none.  alibi_slopes: DEVICE pointer to Hq floats or NULL; adds slope[h]*(j - i) to
 * the scaled score. */
typedef struct { int causal; int window; const float* alibi_slopes; } af_mask;

int         attnfuse_version(void);   /* 100 x major + minor: 110 adds the variant, one-pass backward and fp8 entries */
const char* attnfuse_strerror(af_status st);

/* ---- tuning options ---------------------------------------------------------------------------------
 * Process-wide switches between kernel variants that compute the same result (Section 3.2 makes such choices
 * compile-time constants of the generated kernel; here they select among pre-built instantiations).  Each
 * option starts from the environment variable named beside it, read once when the library first needs an
 * option, else from its default; afterwards only attnfuse_set_option changes it.  Launches read the table,
 * not the environment.  Setting an option while calls are in flight on other host threads affects only
 * calls that start later.  attnfuse_set_option returns AF_ERR_SPEC for an unknown option;
 * attnfuse_get_option returns -1 for one. */
typedef enum {
    AF_OPT_FWD_QTILES = 0,     /* AF_FWD_NQ, default 2: query tiles per CTA of the forward kernel (1 or 2) */
    AF_OPT_FWD_PAIR_HEADS = 1, /* AF_FWD_PAIR, default 1: with an even GQA group the two query tiles of a CTA are two
                                  heads of one kv head; 0: two consecutive row blocks of one head */
    AF_OPT_FWD_KEYS_BF16 = 2,  /* AF_FWD_KEYS_BF16, default 0: key tiles rotated in packed bf16 arithmetic (faster,
                                  about 1.4 times the rounding error on rotated keys; forward only) */
    AF_OPT_BS_ROWPAIR = 3,     /* AF_BS_ROWPAIR, default 1: block-sparse forward with an odd GQA group gives a CTA two
                                  row blocks of one head when the caller supplied pair lists */
    AF_OPT_BWD_ONEPASS = 4,    /* AF_BWD_ONEPASS, default 1: where the one-pass sequence of attnfuse_bwd applies (workspace
                                  of attnfuse_bwd_onepass_workspace_bytes) it is taken where it measured faster: always at
                                  D = 64, at D = 128 when rows are short (at most 12 kept key tiles per query tile on
                                  average, and not over block lists); 2: whenever it applies; 0: never - always the two-kernel sequence, whose dQ is
                                  bit-reproducible */
    AF_OPT_FWD_ALIBI_MMA = 5,  /* AF_FWD_ALIBI_MMA, default 1: the forward kernel adds the ALiBi term slope (j - i) with one
                                  more K step of the score product (the slope split into two bf16 values, the key column
                                  exact in bf16) instead of one fused multiply-add per score in the softmax warps - in the kernels that rotate
                                  on chip, where it measured faster; 2: in every forward kernel; 0: never.  Not used by the additive_bias / relu_attention variants nor together with
                                  AF_OPT_FWD_KEYS_BF16 (no shared memory left for the two small operand tiles) */
    AF_OPT_COUNT_ = 6
} af_option;
af_status attnfuse_set_option(af_option option, int value);
int       attnfuse_get_option(af_option option);

/* ---- device status (bounded waits) ------------------------------------------------------------------
 * Every wait inside the kernels (on an mbarrier) gives up after about one second of SM clocks.  The kernel
 * then records (wait-site code << 16 | low bits of the CTA index) in a status word of the current device,
 * raises a CTA-wide flag that releases the CTA's other waits, frees its tensor memory and returns; the
 * outputs of that launch are undefined and the context stays usable.  No entry point reports the word by
 * itself: poll it with one of the two calls below (e.g. once per step).  Both return AF_OK or
 * AF_ERR_DEVICE_TIMEOUT, store the raw word in *detail (HOST, nullable) and clear it when it was set.
 *   attnfuse_device_status  synchronises the whole device first.
 *   attnfuse_stream_status  reads the word in stream order on `cuda_stream` and synchronises only that
 *                           stream: it sees every launch enqueued on the stream before the call.
 * Neither may be called while a stream capture is in progress (they synchronise). */
af_status attnfuse_device_status(unsigned int* detail);
af_status attnfuse_stream_status(void* cuda_stream, unsigned int* detail);

/* Self-test of that path (for tests and bring-up; no counterpart in the paper): launches one small CTA in which
 * one warp waits, with a limit of `limit_cycles` SM clocks (1e3 .. 1e8), on a barrier that nothing ever
 * arrives on, and a second warp waits on it with the normal limit.  The first wait runs out and records
 * wait-site code 0x7e; the flag it raises releases the second warp; the kernel returns normally.  Afterwards
 * attnfuse_stream_status / attnfuse_device_status report AF_ERR_DEVICE_TIMEOUT once, then AF_OK. */
af_status attnfuse_selftest_wait_timeout(unsigned int limit_cycles, void* cuda_stream);

/* ---- cos/sin table (set-up step of Section 4.1; cached by the caller) --------------------------
 * table: S * rotary_dim/2 pairs of fp32 {cos, sin}(p * theta^(-2i/rotary_dim)), p = pos_offset + s,
 * row-major [S][rotary_dim/2]; angles are formed in fp64 before rounding.  One extra trailer row
 * holds the row-to-row step constants the fused kernels use.  Behind these rows (at the next multiple
 * of 256 bytes) the buffer carries a bf16 copy, S rows of [rotary_dim/2 cos | rotary_dim/2 sin], for
 * the forward kernel's optional packed-bf16 key rotation (environment switch AF_FWD_KEYS_BF16=1:
 * faster, about 1.4 times the rounding error on rotated keys; forward only, off by default).
 * attnfuse_rope_table_bytes returns the size the caller must provide (0 when rotary_dim = 0). */
size_t    attnfuse_rope_table_bytes(int S, int rotary_dim);
af_status attnfuse_rope_table(const af_rope* rope, int S, void* table, void* cuda_stream);

/* ---- separate RoPE pass (the pre-rotation arm of Section 5.3) -----------------------------------
 * Rotates every row of x_in [B, n_heads, S, D] (contiguous) into x_out (may alias x_in).
 * inverse != 0 applies the transpose rotation.  shape->Hq/Hkv are ignored; n_heads is used. */
af_status attnfuse_rope(const af_shape* shape, int n_heads, const void* x_in, void* x_out,
                        const af_rope* rope, const void* rope_table, int inverse, void* cuda_stream);

/* ---- fused forward (Sections 2, 4.1) ---------------------------------------------------------------
 * One kernel: rotate Q and K tiles on chip, S = Q'K'^T, scale, ALiBi, mask, online softmax, O = P V.
 * q [B,Hq,S,D], k, v [B,Hkv,S,D] bf16 with strides sq / skv (NULL = contiguous).
 * rope_table: from attnfuse_rope_table for the same (rope, S); may be NULL iff rotary_dim = 0.
 * o: [B,Hq,S,D] contiguous, o_dtype AF_BF16 or AF_F32.
 * lse: [B,Hq,S] fp32, L = m + ln(l) (Section 4.4), natural log; nullable. */
af_status attnfuse_fwd(const af_shape* shape, const void* q, const void* k, const void* v,
                       const af_strides* sq, const af_strides* skv,
                       const af_rope* rope, const void* rope_table, const af_mask* mask,
                       int gqa_group, float softmax_scale,
                       void* o, af_dtype o_dtype, float* lse, void* cuda_stream);

/* ---- hybrid arm of Section 5.3: rotate K once, fuse only the Q rotation -------------------------------
 * Same result as attnfuse_fwd (up to the bf16 rounding of a few rotated elements).  A RoPE pass writes
 * K' = RoPE(K) into the workspace (contiguous [B,Hkv,S,D] bf16), then the forward kernel runs with the
 * on-chip rotation of key tiles switched off and the query tiles still rotated on chip.  With grouped
 * queries K is the small operand (Hkv heads against Hq), so rotating it once costs little HBM traffic
 * and spares every CTA the rotation of each key tile it streams.  rotary_dim = 0: plain attnfuse_fwd.
 * workspace (device): attnfuse_fwd_hybrid_workspace_bytes(shape) bytes, 16-byte aligned, caller-owned;
 * AF_ERR_WORKSPACE when missing or too small. */
size_t    attnfuse_fwd_hybrid_workspace_bytes(const af_shape* shape);
af_status attnfuse_fwd_hybrid(const af_shape* shape, const void* q, const void* k, const void* v,
                              const af_strides* sq, const af_strides* skv,
                              const af_rope* rope, const void* rope_table, const af_mask* mask,
                              int gqa_group, float softmax_scale,
                              void* o, af_dtype o_dtype, float* lse,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---- block-sparse attention (Section 4.3) ------------------------------------------------------------
 * The caller evaluates its block predicate once and passes the active 128 x 128 blocks as index lists
 * (device memory, int32): by query row block (CSR: row_ptr [nb + 1], col_idx [row_ptr[nb]], nb = ceil(S/128))
 * and, for the backward, by key block (CSC: col_ptr [nb + 1], row_idx [col_ptr[nb]]).  Kernels visit only
 * the listed blocks, so the work is proportional to the active fraction.  A pair (i, j) is kept iff its
 * block is listed AND the element mask of af_mask keeps it (so listing a diagonal block under a causal
 * mask gives the usual triangle); a query row without a kept pair gets O = 0, L = -inf, zero gradients.
 * The lists are not validated on the device: indices must lie in [0, nb) and the CSC lists must describe
 * the same set of blocks as the CSR lists. */
typedef struct {
    int block;            /* block edge; must be 128 */
    const int* row_ptr;   /* CSR by query row block (device) */
    const int* col_idx;
    const int* col_ptr;   /* CSC by key block (device); needed by attnfuse_bwd_blocks only */
    const int* row_idx;
    const int* row_order; /* optional (NULL = 0, 1, 2, ...): the query row blocks in the order in which CTAs should be
                             launched, normally by decreasing list length so that the longest lists start first */
    const int* col_order; /* the same for key blocks (dK/dV kernel of the backward) */
    /* Optional (all three NULL = not given), used by attnfuse_fwd_blocks when the GQA group is odd, where no two
     * query heads share K and V: lists by PAIR of query row blocks (2r, 2r + 1), so that one CTA can work on two
     * row blocks of a head at once.  pair_ptr [ceil(nb/2) + 1]; pair_idx: per pair the sorted union of the two
     * row blocks' lists, each entry = key block | (1 << 28 if row block 2r lists it) | (1 << 29 if 2r + 1 does);
     * pair_order: optional launch order of the pairs (NULL = 0, 1, 2, ...). */
    const int* pair_ptr;
    const int* pair_idx;
    const int* pair_order;
} af_blocks;

/* attnfuse_fwd over the listed blocks. */
af_status attnfuse_fwd_blocks(const af_shape* shape, const void* q, const void* k, const void* v,
                              const af_strides* sq, const af_strides* skv,
                              const af_rope* rope, const void* rope_table, const af_mask* mask,
                              int gqa_group, float softmax_scale, const af_blocks* blocks,
                              void* o, af_dtype o_dtype, float* lse, void* cuda_stream);

/* ---- forward with 8-bit operands (opt-in; Section 9.1 names fp8 tensor cores as the natural extension) ----
 * q8 [B,Hq,S,D], k8 [B,Hkv,S,D]: E4M3 codes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities),
 * contiguous; vt8 [B,Hkv,D,S]: the E4M3 codes of V TRANSPOSED (keys contiguous); all DEVICE, 16-byte aligned.
 * A value is code x scale: scale_q, scale_k, scale_v > 0 are per-tensor dequantisation scales (HOST floats).
 * Computes softmax(softmax_scale x (q k^T) + mask) v with both products on the fp8 tensor path (fp32 accumulation),
 * the softmax in fp32 and the probabilities rounded to E4M3 before the second product (the row sum uses the unrounded
 * ones).  No rotation is applied: rotate in bf16 (attnfuse_rope) and quantise afterwards.  mask: causal and window as
 * in attnfuse_fwd; ALiBi slopes -> AF_ERR_SPEC.  D = 128 and S a multiple of 16 (AF_ERR_SHAPE otherwise).
 * o [B,Hq,S,D] in o_dtype, lse (nullable) [B,Hq,S] as in attnfuse_fwd.  Precision: the products of 8-bit operands are
 * exact in fp32, so L matches the definition to fp32 rounding; the E4M3 rounding of a probability is up to 2^-4
 * relative, and outputs are held to max abs 1e-1 and mean abs 8e-3 against the fp64 oracle evaluated on the
 * dequantised inputs (unit-variance data; measured max 0.05, mean 0.001-0.006) - a bound of its own, not the bf16 path's. */
af_status attnfuse_fwd_fp8(const af_shape* shape, const void* q8, const void* k8, const void* vt8,
                           const af_mask* mask, int gqa_group, float softmax_scale,
                           float scale_q, float scale_k, float scale_v,
                           void* o, af_dtype o_dtype, float* lse, void* cuda_stream);

/* ---- composed variants (Section 3.1: the ten combinators) ---------------------------------------------
 * One description of a variant and one forward entry point for it, the counterpart of a program composed
 * from the paper's combinators (Section 3.1) and run through its single run-time entry (Section 3.3):
 *   scaled_dot_product  -> softmax_scale        rope            -> rope + rope_table
 *   causal              -> mask.causal          sliding_window  -> mask.window
 *   full                -> mask.causal = 0 and mask.window < 0 (nothing masked)
 *   block_sparse        -> blocks               alibi           -> mask.alibi_slopes
 *   additive_bias       -> bias                 softmax / relu_attention -> normaliser
 * additive_bias: a dense fp32 tensor bias[bb, hh, i, j] (DEVICE, contiguous [bias_B, bias_H, S, S], 4-byte
 * aligned; extents 1 = broadcast, else B resp. Hq), added to the scaled score after the softmax scale, like
 * the ALiBi term.  A bias of -inf drops the pair like a mask.  NULL: none.  The kernel reads it with plain
 * loads, one row of 128 values per thread and key tile (16-byte loads when S is a multiple of 4): the
 * variant is bound by the S x S bias traffic, not by the tensor pipe.
 * relu_attention (the paper names the combinator only; reading): P_ij = max(s_ij, 0) / n_i over the kept
 * pairs, n_i = number of kept pairs of row i (pairs that the mask keeps and whose bias is finite), in place
 * of the softmax; there is no log-sum-exp: with relu_attention `lse` (nullable) receives n_i as a float, the
 * row statistic that attnfuse_bwd_variant needs; not available over block lists.
 * Errors as for attnfuse_fwd; AF_ERR_SHAPE for bias extents other than 1 / B / Hq, AF_ERR_SPEC for an
 * unknown normaliser and for relu_attention with blocks.
 *
 * attnfuse_bwd_variant: the backward of the same description.  Arguments as attnfuse_bwd; `lse` is what the
 * forward of the SAME variant wrote (L, or n_i under relu_attention).  No gradient flows into the bias.  With
 * relu_attention dS_ij = [s_ij > 0] dP_ij / n_i.  A variant without bias and with the softmax normaliser takes
 * the sequences of attnfuse_bwd / attnfuse_bwd_blocks.  With a bias or relu_attention: dense only (AF_ERR_SPEC
 * with blocks), always the two-kernel sequence (deterministic), and with a rotation the workspace must hold
 * delta and both rotated caches (attnfuse_bwd_workspace_bytes; AF_ERR_WORKSPACE otherwise); the first query
 * rows get no fp32 treatment there (see attnfuse_bwd), so rows with a handful of keys carry the bf16 roundings
 * of P and dS at full size. */
typedef enum { AF_NORM_SOFTMAX = 0, AF_NORM_RELU = 1 } af_normaliser;
typedef struct {
    af_rope rope;
    const void* rope_table;      /* from attnfuse_rope_table; may be NULL iff rope.rotary_dim = 0 */
    af_mask mask;
    const float* bias;           /* additive_bias or NULL */
    int bias_B, bias_H;          /* its batch and head extents: 1 or B, 1 or Hq */
    af_normaliser normaliser;
    const af_blocks* blocks;     /* block_sparse lists or NULL (dense) */
} af_variant;
af_status attnfuse_bwd_variant(const af_shape* shape, const void* q, const void* k, const void* v,
                               const void* o, const float* lse, const void* d_o,
                               const af_strides* sq, const af_strides* skv, const af_variant* variant,
                               int gqa_group, float softmax_scale,
                               void* dq, af_dtype dq_dtype, void* dk, void* dv, af_dtype dkv_dtype,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);
af_status attnfuse_fwd_variant(const af_shape* shape, const void* q, const void* k, const void* v,
                               const af_strides* sq, const af_strides* skv, const af_variant* variant,
                               int gqa_group, float softmax_scale,
                               void* o, af_dtype o_dtype, float* lse, void* cuda_stream);

/* Same computation with HOST buffers: q, k, v, o (bf16) and lse (nullable) are host pointers
 * (pinned memory: with pageable memory the copies are not asynchronous).  `staging` is a DEVICE buffer
 * of at least attnfuse_fwd_host_staging_bytes() bytes, caller-owned.  The work is cut into chunks of
 * consecutive (batch element, kv head) units and pipelined: host-to-device copies on the caller's stream,
 * the kernels and the device-to-host copies on two internal streams of the library (created once per
 * device), so that the two copy directions and the kernels overlap; the caller's stream waits for the
 * last result at the end of the call, so work enqueued on it afterwards sees o_host and lse_host complete
 * and may reuse `staging`.  Results are bit-identical to attnfuse_fwd on the same data.  Calls are
 * serialised on the host by a lock.  alibi slopes inside `mask` remain a DEVICE pointer. */
size_t    attnfuse_fwd_host_staging_bytes(const af_shape* shape);
af_status attnfuse_fwd_host(const af_shape* shape, const void* q_host, const void* k_host, const void* v_host,
                            const af_rope* rope, const void* rope_table, const af_mask* mask,
                            int gqa_group, float softmax_scale,
                            void* o_host, float* lse_host, void* staging, size_t staging_bytes,
                            void* cuda_stream);

/* ---- Flash Decoding (Section 4.2; Table "Flash Decoding") ---------------------------------------------
 * One query position per head (the last one, N - 1) against a KV cache of N = shape->S keys:
 *   o[b,h,:] = softmax_j( c * <q[b,h], k[b,h/g,j]> + m_h (j - (N - 1)) ) v[b,h/g,j],  j kept iff j >= N - 1 - W.
 * Phase 1 splits the cache over n_splits CTAs per (batch, kv head); each computes a partial (max, sum,
 * accumulator) for the g query heads of its kv head (packed as rows of one MMA tile, K and V read once);
 * phase 2 merges the partials with a log-sum-exp (same launch, see `workspace` below).  No rotation is applied: q and the cached keys are used
 * as they are (a cache holds rotated keys; rotate q with attnfuse_rope).  mask->causal is ignored (every
 * cached key precedes the query); window and ALiBi slopes apply as in attnfuse_fwd.
 * q, o: [B,Hq,D] bf16 contiguous (device); k, v: [B,Hkv,N,D] bf16 with strides skv (NULL = contiguous; the
 * rows need 16-byte alignment and strides that are multiples of 8 elements); lse (nullable): [B,Hq] fp32.
 * gqa_group <= 16; D in {64, 128}.  n_splits <= 0: attnfuse_decode_splits(shape), the largest count that keeps the
 * grid of n_splits x B x Hkv CTAs within one CTA per SM of the current device (one wave) with at least 128 keys
 * per split.  Larger requests are clamped to ceil(S / 128) and to 256 splits.
 * workspace: attnfuse_decode_workspace_bytes(shape, n_splits) device bytes: a ticket counter per (batch, kv head)
 * at its head, then the partials.  Both phases run in ONE launch: the CTA that finishes last for a kv head merges
 * that head group's partials (in split order: the result does not depend on which CTA is last).  The counters must
 * be ZERO before the first call that uses a workspace - call attnfuse_decode_workspace_init once after allocating it
 * (it clears the workspace on the given stream) - and every call leaves them zero.  A workspace serves one call at
 * a time: calls that may overlap on the GPU need workspaces of their own.  After AF_ERR_DEVICE_TIMEOUT, clear it again. */
int       attnfuse_decode_splits(const af_shape* shape);
size_t    attnfuse_decode_workspace_bytes(const af_shape* shape, int n_splits);
af_status attnfuse_decode_workspace_init(void* workspace, size_t workspace_bytes, void* cuda_stream);
af_status attnfuse_decode(const af_shape* shape, const void* q, const void* k, const void* v,
                          const af_strides* skv, const af_mask* mask, int gqa_group, float softmax_scale,
                          void* o, float* lse, int n_splits,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---- fused backward (Section 4.4) -------------------------------------------------------------------
 * Row-reduced gradients delta = rowsum(dO * O); dK/dV accumulation per key tile; dQ accumulation per
 * query tile.  Probabilities are recomputed from lse; the rotation is recomputed and gradients w.r.t.
 * rotated rows are rotated back in the epilogues.
 * o, d_o: [B,Hq,S,D] bf16 contiguous; lse from the forward.
 * dq [B,Hq,S,D] (dq_dtype), dk, dv [B,Hkv,S,D] (dkv_dtype), contiguous; dk/dv sum over the group.
 * workspace: attnfuse_bwd_workspace_bytes(shape) bytes hold delta (4 bytes per query row, rounded up to
 * 256), a cache of the rotated K (B*Hkv*S*D bf16) and a cache of the rotated Q (B*Hq*S*D bf16), in this
 * order.  With all three, K is rotated once by a RoPE pass, each Q tile once by the dQ kernel that owns it
 * (which also writes it to the cache), and the dK/dV kernel runs last without rotating anything in its
 * loop.  A smaller workspace is accepted: with delta + K cache the dK/dV kernel runs first, rotates K once
 * per key tile and every Q tile it streams, and the dQ kernel streams the cached K; with delta alone both
 * kernels rotate everything they touch on chip.  Results of the three set-ups agree up to the bf16
 * rounding of a few rotated elements.  These three are deterministic: no atomics, every accumulator has one
 * owner and a fixed order of additions.
 * One-pass sequence (dense masks and block lists): with a workspace of attnfuse_bwd_onepass_workspace_bytes(shape) -
 * the three pieces above followed by an fp32 accumulator of dQ (B*Hq*S*D*4 bytes) - and where option
 * AF_OPT_BWD_ONEPASS selects it, RoPE passes write both caches and ONE kernel per key tile forms dK, dV and its
 * share of dQ (five tile products per kept tile pair instead of seven; S and dP are not recomputed a second
 * time).  The shares of dQ from different key tiles are added into the accumulator with fp32 reductions in
 * global memory, in an order that depends on CTA scheduling: dQ may differ in its last bits from run to run
 * (within the same bounds against the exact result); dK and dV stay reproducible.  A last pass scales the
 * accumulator, rotates it back and writes dq.  The accumulator needs no initialisation by the caller. */
size_t    attnfuse_bwd_workspace_bytes(const af_shape* shape);
size_t    attnfuse_bwd_onepass_workspace_bytes(const af_shape* shape);
af_status attnfuse_bwd(const af_shape* shape, const void* q, const void* k, const void* v,
                       const void* o, const float* lse, const void* d_o,
                       const af_strides* sq, const af_strides* skv,
                       const af_rope* rope, const void* rope_table, const af_mask* mask,
                       int gqa_group, float softmax_scale,
                       void* dq, af_dtype dq_dtype, void* dk, void* dv, af_dtype dkv_dtype,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/* attnfuse_bwd over the listed blocks (Section 4.3); needs both the CSR and the CSC lists of `blocks`.
 * lse must come from attnfuse_fwd_blocks with the same lists; rows whose L is -inf get zero gradients. */
af_status attnfuse_bwd_blocks(const af_shape* shape, const void* q, const void* k, const void* v, const void* o,
                              const float* lse, const void* d_o,
                              const af_strides* sq, const af_strides* skv,
                              const af_rope* rope, const void* rope_table, const af_mask* mask,
                              int gqa_group, float softmax_scale, const af_blocks* blocks,
                              void* dq, af_dtype dq_dtype, void* dk, void* dv, af_dtype dkv_dtype,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---- backward without a caller workspace (the paper has no counterpart) ---------------------------
 * Some callers are not allowed to obtain device memory at the point where they need the backward:
 * a plug-in that runs inside another framework's enqueue hook, a serving loop whose memory pool was
 * frozen at start-up, code that runs while the allocator is locked by someone else.  For them this
 * variant of attnfuse_bwd keeps the one piece of scratch the backward needs (delta, one fp32 per
 * query row) in a fixed array inside the library instead of a caller workspace.  Inputs and outputs
 * are still the caller's, exactly as for attnfuse_bwd.  The call always runs the delta-only set-up of
 * attnfuse_bwd (both gradient kernels rotate what they touch on chip, nothing else is cached), whatever
 * the problem size: its results are bit-identical to attnfuse_bwd given a workspace of exactly
 * 4 * B*Hq*S bytes rounded up to 256, and equal to attnfuse_bwd with a full workspace up to the bf16
 * rounding of a few rotated elements.
 *
 *  - Limit: B*Hq*S <= AF_BWD_STATIC_MAX_ROWS (4 MiB of scratch, which every GPU that loads the library
 *    holds until the process exits).  Larger problems return AF_ERR_STATIC_LIMIT and launch nothing.
 *  - The call allocates and frees nothing, on the host side of CUDA or through any library.
 *  - The first call on each device looks up the device address of the array (with that device
 *    current) and remembers it; make that first call outside any stream capture.
 *  - All calls on a device share the array and it keeps whatever the previous call left there.  Nothing
 *    in it has to start at zero (each call overwrites the part it reads), but two calls that overlap
 *    on the GPU (different streams, no ordering between them) race on it: order them. */
#define AF_BWD_STATIC_MAX_ROWS (1 << 20)
af_status attnfuse_bwd_static(const af_shape* shape, const void* q, const void* k, const void* v,
                              const void* o, const float* lse, const void* d_o,
                              const af_strides* sq, const af_strides* skv,
                              const af_rope* rope, const void* rope_table, const af_mask* mask,
                              int gqa_group, float softmax_scale,
                              void* dq, af_dtype dq_dtype, void* dk, void* dv, af_dtype dkv_dtype,
                              void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* ATTNFUSE_H_ */
