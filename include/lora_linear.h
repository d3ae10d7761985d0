/*
 * lora_linear.h - C ABI of the B200 (sm_100a) LoRA projection layer, forward and backward.
 *
 * The layer is the low-rank-adapter form of a decoder projection with a frozen weight
 * (Section 3.2.2, LoRA fine-tuning; adapter rank r and alpha as in Section 4.5, scale = alpha / r):
 *
 *     forward    Y  = X W^T + scale (X A^T) B^T
 *     backward   dX = dY W + scale (dY B) A
 *                dB = scale dY^T (X A^T)
 *                dA = scale (dY B)^T X
 *
 * Layouts: every tensor is dense row-major, last index contiguous.
 *     X [T, d_in]  W [d_out, d_in]  A [r, d_in]  B [d_out, r]  Y, dY [T, d_out]  dX [T, d_in]   bf16
 *     dA [r, d_in]  dB [d_out, r]                                                                   fp32
 * T is the number of packed trajectory tokens of the batch; packing boundaries do not reach a
 * projection layer, so no sequence offsets are passed.
 *
 * Conventions
 *   - Every function returns an int: LORA_OK (0) or a negative lora_status_t.  Nothing throws,
 *     nothing calls exit().
 *   - Tensor pointers are DEVICE pointers owned by the caller (unless a parameter is named h_*),
 *     16-byte aligned.  Inputs are read-only; outputs are overwritten.  The one exception is opt-in per plan:
 *     after lora_plan_set_grad_accumulation(plan, 1) the backward calls ADD to dA and dB (dX is still overwritten).
 *     No output may alias an input or another output.
 *   - d_in and d_out must be multiples of 8; r a multiple of 8 with 8 <= r <= 64; T >= 0.
 *   - `stream` is a cudaStream_t passed as void*.  Calls only enqueue work and return; they do not
 *     synchronise.  A plan must not be used from two host threads, or on two streams, at once.
 *     The forward and backward calls (plain, saved-P, grouped, NF4, dense dW) therefore work under stream capture: a step
 *     captured into a CUDA graph replays bit-identically (what a launch-bound batch of a few hundred tokens wants).
 *     Not capturable: lora_last_device_status, lora_plan_last_gemm_clock and lora_grad_contract_noalloc_status, which
 *     synchronise the stream and copy to the host.
 *   - The library never allocates device memory except one 256-byte status word block per plan;
 *     scratch is caller-provided (lora_plan_set_workspace): backward always needs it, forward needs it whenever the
 *     selector chose the K-extended form (cfg.fwd_ext; lora_plan_workspace_bytes reports fwd_bytes > 0 then).
 *   - There is no CPU fallback: without a CUDA device of compute capability 10.x the calls fail
 *     with LORA_ERR_NO_DEVICE.
 */
#ifndef LORA_LINEAR_H_
#define LORA_LINEAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum lora_status {
  LORA_OK = 0,
  LORA_ERR_INVALID_ARG = -1,       /* null pointer, negative size, bad buffer length            */
  LORA_ERR_UNSUPPORTED_SHAPE = -2, /* d_in/d_out not multiples of 8, r outside {8,16,...,64}     */
  LORA_ERR_MISALIGNED = -3,        /* a tensor pointer is not 16-byte aligned                    */
  LORA_ERR_WORKSPACE = -4,         /* backward called without (enough) workspace                 */
  LORA_ERR_CUDA = -5,              /* a CUDA runtime / driver call failed (launch, descriptor)   */
  LORA_ERR_DEVICE_TIMEOUT = -6,    /* a bounded device-side wait ran out (lora_last_device_status)*/
  LORA_ERR_NO_DEVICE = -7          /* no usable sm_100 device                                    */
} lora_status_t;

typedef struct lora_plan lora_plan_t; /* opaque, host memory owned by the library */

typedef struct lora_shape {
  int64_t T;     /* tokens (rows of X, Y, dY, dX) */
  int64_t d_in;  /* input features                */
  int64_t d_out; /* output features               */
  int64_t r;     /* adapter rank                  */
} lora_shape_t;

/* What the per-shape selector chose (Section 3.2.2 "dynamic profiling" analogue at kernel level). */
typedef struct lora_kernel_config {
  int32_t block_m;         /* token rows per GEMM tile: 128 (one CTA) or 256 (CTA pair)        */
  int32_t fwd_block_n;     /* output columns per tile of the forward GEMM (multiple of 16)     */
  int32_t dx_block_n;      /* output columns per tile of the dX GEMM                           */
  int32_t block_k;         /* contraction elements per pipeline stage (64)                     */
  int32_t stages;          /* depth of the TMA -> MMA shared-memory ring, forward GEMM         */
  int32_t group_m;         /* tile rasterisation: m-tiles per band (L2 reuse)                  */
  int32_t split_k;         /* k-splits per tile of the forward GEMM (1 = none)                 */
  int32_t r_pad;           /* rank padded to the MMA granularity (multiple of 16)              */
  int32_t fwd_ctas;        /* persistent CTAs of the forward GEMM                              */
  int32_t dx_ctas;         /* persistent CTAs of the dX GEMM                                   */
  int32_t tail_delay;      /* k-blocks of the next tile issued before a tile's rank-r MMA      */
  int32_t grad_feat_chunk; /* features per CTA of the adapter-gradient kernels                 */
  int32_t grad_stages;     /* ring depth of the adapter-gradient kernels                       */
  int32_t da_feat_chunks;  /* dA kernel grid: feature chunks x token chunks (one cluster each) */
  int32_t da_token_chunks;
  int32_t db_feat_chunks;  /* dB kernel grid                                                   */
  int32_t db_token_chunks;
  int32_t db_feat_chunk;   /* features per CTA of the dB kernel (grad_feat_chunk is dA's)      */
  int32_t cta_group;       /* 1: one CTA per tile; 2: two CTAs (one TPC) share a 256-row tile  */
  int32_t dx_stages;       /* ring depth of the dX GEMM                                        */
  int32_t prefetch_dist;   /* k-blocks by which L2 prefetches run ahead of the ring (0: unused)*/
  int32_t db_stages;       /* ring depth of the dB kernel (grad_stages is dA's)                */
  int32_t q_feat_chunk;    /* Q = dY B pre-pass (CTA-pair backward): features per CTA, grid, ring depth */
  int32_t q_feat_chunks;
  int32_t q_token_chunks;
  int32_t q_stages;
  int32_t dx_split_k;      /* k-splits per tile of the dX GEMM                                           */
  int32_t fwd_ext;         /* 1: forward runs as X A^T pre-pass + K-extended GEMM (needs the workspace)  */
  int32_t bwd_merged;      /* 1: lora_linear_bwd = [dY B + X A^T in one launch] dX GEMM [dA + dB in one launch];      */
                           /* 0: dY B | dX GEMM | dA (+ X A^T) | dB, one launch each                                  */
  int32_t pair_feat_chunk; /* the dA + dB launch of the merged form: features per CTA, feature chunks of both, cluster */
  int32_t pair_feat_chunks;
  int32_t pair_token_chunks;
  int32_t da_with_p;       /* split form: 1: X A^T is recomputed inside the dA launch; 0: in its own skinny pass over X */
  int32_t dan_feat_chunk;  /* dA launch without X A^T (saved-P backward, or da_with_p = 0): features per CTA, grid    */
  int32_t dan_feat_chunks;
  int32_t dan_token_chunks;
  int32_t dbq_feat_chunk;  /* dB launch that also computes dY B (saved-P backward): features per CTA, grid            */
  int32_t dbq_feat_chunks;
  int32_t dbq_token_chunks;
  int32_t dw_block_n;      /* dense weight gradient GEMM (lora_dense_dw): d_in columns per tile,         */
  int32_t dw_split_k;      /*   splits along the tokens, persistent CTAs                                 */
  int32_t dw_ctas;
} lora_kernel_config_t;

/* Host-only: run the tile / split selector for a shape on a device with `num_sms` SMs.
 * Needs no GPU.  Returns LORA_ERR_UNSUPPORTED_SHAPE for shapes the kernels do not cover. */
int lora_select_config(const lora_shape_t* shape, int num_sms, lora_kernel_config_t* out);

/* Host-only: bytes of scratch lora_linear_bwd needs for a shape.  The forward uses the same scratch when the selector
 * picks its K-extended form for the shape (lora_kernel_config_t.fwd_ext = 1, e.g. every 4096-wide or wider output
 * from 4096 tokens on); the fused form needs none.  lora_plan_workspace_bytes reports both figures for a plan. */
int lora_workspace_bytes(const lora_shape_t* shape, int num_sms, size_t* bwd_bytes);

/* Create / destroy a plan for one shape on CUDA device `device` (runs the selector, allocates the
 * 256-byte device status block).  The plan is host memory owned by the library.
 * With the environment variable LORA_LOG=1 every new plan prints one line to stderr with what the selector chose
 * (the text lora_plan_describe returns). */
int lora_plan_create(const lora_shape_t* shape, int device, lora_plan_t** out);
int lora_plan_destroy(lora_plan_t* plan);

/* Scratch sizes of a plan; either pointer may be NULL.  fwd_bytes is 0 unless the selector chose the K-extended
 * forward (cfg.fwd_ext), which uses the same workspace as backward. */
int lora_plan_workspace_bytes(const lora_plan_t* plan, size_t* fwd_bytes, size_t* bwd_bytes);

/* Register caller-owned device scratch (256-byte aligned, at least bwd_bytes).  The memory stays
 * owned by the caller and must outlive every backward call that uses the plan. */
int lora_plan_set_workspace(lora_plan_t* plan, void* dev_ptr, size_t bytes);

/* Gradient accumulation over micro-batches (the paper trains with global batches of 32-96 sequences, i.e. several
 * backward passes per optimiser step): with `enable` != 0 every backward call on the plan ADDS its dA and dB to the
 * caller's buffers instead of overwriting them (dA += ..., dB += ...; the caller zeroes them before the first
 * micro-batch).  The sum stays deterministic: old value + the call's partial sums in their fixed order.  dX is always
 * overwritten.  Off by default. */
int lora_plan_set_grad_accumulation(lora_plan_t* plan, int enable);

/* Copy the selector's choice / a one-line description into caller memory. */
int lora_plan_get_config(const lora_plan_t* plan, lora_kernel_config_t* out);
int lora_plan_describe(const lora_plan_t* plan, char* buf, size_t n);

/* Forward:  Y = X W^T + scale (X A^T) B^T.
 * TMA-staged bf16 tiles, tcgen05 MMA into TMEM.  Two forms, chosen per shape (cfg.fwd_ext):
 *   fused       one kernel; X A^T rides the main loop as extra accumulator columns and the rank-r product is one more
 *               MMA group before the epilogue (narrow outputs, small batches; needs no workspace);
 *   K-extended  a skinny pass over X produces scale (X A^T)^T, which then enters the GEMM as one more k-block, so that
 *               every MMA column is an output column (wide outputs, large ranks, >= 4096 tokens; needs the workspace:
 *               LORA_ERR_WORKSPACE otherwise, see lora_plan_workspace_bytes). */
int lora_linear_fwd(lora_plan_t* plan, const void* X, const void* W, const void* A, const void* B,
                    float scale, void* Y, void* stream);

/* Backward:  dX = dY W + scale (dY B) A,  dA = scale (dY B)^T X,  dB = scale dY^T (X A^T).
 * Does not depend on a preceding forward call (X A^T is recomputed).  Needs the workspace.
 * dA and dB are fp32 and are overwritten.
 * Launches (cfg.bwd_merged = 1, the default): dY B and X A^T side by side in one skinny launch, the dX GEMM, dA and dB side
 * by side in one skinny launch.  (cfg.bwd_merged = 0: dY B pre-pass, dX GEMM, dA with X A^T riding along or preceded by
 * its own pass over X, dB.)  No launch only finishes another's sums: dA and dB are added up over the token chunks inside thread-block clusters, the
 * skinny products over feature chunks by the last CTA to arrive, both in a fixed order (bitwise reproducible). */
int lora_linear_bwd(lora_plan_t* plan, const void* dY, const void* X, const void* W, const void* A,
                    const void* B, float scale, void* dX, void* dA, void* dB, void* stream);

/* Backward that reuses the forward's X A^T (what an autograd function would stash): valid only directly after a
 * lora_linear_fwd call on the SAME plan with the same X, A and scale, made while the workspace was registered (the
 * forward then leaves scale (X A^T)^T, 2 r_pad bytes per token, in the workspace).  Same results as lora_linear_bwd
 * up to rounding order; one pass over dY and one over X instead of three skinny passes: the dB kernel also produces
 * scale (dY B)^T, the dX GEMM and the dA kernel consume it.  Returns LORA_ERR_INVALID_ARG when no matching forward
 * result is held.  For batches of at most 128 tokens it is the same as lora_linear_bwd. */
int lora_linear_bwd_saved_p(lora_plan_t* plan, const void* dY, const void* X, const void* W, const void* A,
                            const void* B, float scale, void* dX, void* dA, void* dB, void* stream);

/* The three stages of lora_linear_bwd as separate calls, for callers that schedule them themselves.
 * They communicate through the plan's workspace and must run in this order on one stream (or with
 * equivalent event dependencies):
 *   lora_linear_bwd_q    optional: only the skinny pre-pass scale (dY B)^T -> workspace (streams dY once).  The next
 *                        lora_linear_bwd_dx on the plan (same dY, B, scale) then launches the GEMM alone; any other
 *                        backward call on the plan in between discards the staged product.  A no-op for plans with
 *                        T <= 128, whose dX kernel computes dY B itself.
 *   lora_linear_bwd_dx   dX = dY W + scale (dY B) A ; leaves scale (dY B)^T in the workspace
 *   lora_linear_bwd_da   dA = scale (dY B)^T X, streams X once ; leaves scale (X A^T)^T in the workspace
 *   lora_linear_bwd_db   dB = scale dY^T (X A^T), streams dY once
 * `scale` must be the same in all three. */
int lora_linear_bwd_q(lora_plan_t* plan, const void* dY, const void* B, float scale, void* stream);
/* The two skinny launches of the merged form as separate calls (the order is lora_linear_bwd_sides, lora_linear_bwd_dx,
 * lora_linear_bwd_grads, same scale):
 *   lora_linear_bwd_sides   scale (dY B)^T and scale (X A^T)^T -> workspace in ONE launch (streams dY and X once); the next
 *                           lora_linear_bwd_dx on the plan launches the GEMM alone
 *   lora_linear_bwd_grads   dA and dB in ONE launch from the two products in the workspace (streams X and dY once) */
int lora_linear_bwd_sides(lora_plan_t* plan, const void* dY, const void* X, const void* A, const void* B, float scale,
                          void* stream);
int lora_linear_bwd_grads(lora_plan_t* plan, const void* dY, const void* X, const void* A, float scale, void* dA, void* dB,
                          void* stream);
int lora_linear_bwd_dx(lora_plan_t* plan, const void* dY, const void* W, const void* A, const void* B,
                       float scale, void* dX, void* stream);
int lora_linear_bwd_da(lora_plan_t* plan, const void* X, const void* A, float scale, void* dA, void* stream);
int lora_linear_bwd_db(lora_plan_t* plan, const void* dY, float scale, void* dB, void* stream);

/* Grouped projections: G = 2..4 projections that consume the SAME activations X (the attention q/k/v projections, the MLP
 * gate/up projections; Section 4.5 adapts q, k, v, o with lora_r = 32) as one layer call.  Group g has its own frozen
 * W_g [d_g, d_in] and its own adapter A_g [r, d_in], B_g [d_g, r]; all groups share T, d_in, r and scale:
 *
 *     Y_g = X W_g^T + scale (X A_g^T) B_g^T        dX = sum_g ( dY_g W_g + scale (dY_g B_g) A_g )
 *     dA_g = scale (dY_g B_g)^T X                  dB_g = scale dY_g^T (X A_g^T)
 *
 * i.e. exactly what G separate lora_linear_fwd / lora_linear_bwd calls compute, with the G partial dX added up.
 * Operands are the groups' tensors stacked along their row (W, A, B) or column (Y, dY) index, in group order:
 *     W_cat [sum d_g, d_in]   A_cat [G r, d_in]   B_cat [sum d_g, r]   Y_cat, dY_cat [T, sum d_g]     bf16
 *     dX [T, d_in] bf16       dA_cat [G r, d_in]  dB_cat [sum d_g, r]                                  fp32
 * (group g's Y is the column range [off_g, off_g + d_g) of Y_cat, a strided view).  What grouping buys: X is streamed once
 * per stage for all groups; the forward is ONE GEMM over sum d_g output columns (narrow projections such as the 1024-wide
 * k/v no longer leave CTA pairs idle) whose rank-r k-block picks, per output tile, the rows of scale (X A^T)^T and of B
 * that belong to the tile's group; dX is ONE GEMM over the contraction sum d_g plus one rank-r k-block per group; all dY_g B_g
 * and X A_cat^T run in one skinny launch, all dA_g and dB_g in another.  No block of zeros is multiplied and nothing is
 * computed only to be dropped.
 * Limits (LORA_ERR_UNSUPPORTED_SHAPE otherwise; run the projections through their own plans then): T > 128;
 * r in {16, 32, 48, 64}; every d_g a multiple of 256; G + ceil(G r / 64) <= 6.
 * A grouped plan is created by lora_plan_create_grouped and used with the two *_grouped calls only (the plain calls return
 * LORA_ERR_INVALID_ARG on it and vice versa); workspace, wait limit, gradient accumulation, status and destruction go through
 * the same lora_plan_* calls.  Both calls need the workspace (lora_plan_workspace_bytes). */
typedef struct lora_group_shape {
  int64_t T;        /* tokens                                 */
  int64_t d_in;     /* input features, shared                 */
  int64_t r;        /* adapter rank of every group            */
  int32_t n_groups; /* 2 .. 4                                 */
  int64_t d_out[4]; /* output features of each group          */
} lora_group_shape_t;
int lora_plan_create_grouped(const lora_group_shape_t* shape, int device, lora_plan_t** out);
int lora_linear_fwd_grouped(lora_plan_t* plan, const void* X, const void* W_cat, const void* A_cat, const void* B_cat,
                            float scale, void* Y_cat, void* stream);
int lora_linear_bwd_grouped(lora_plan_t* plan, const void* dY_cat, const void* X, const void* W_cat, const void* A_cat,
                            const void* B_cat, float scale, void* dX, void* dA_cat, void* dB_cat, void* stream);

/* Dense weight gradient of full fine-tuning (Section 4.5, "Full-model tuning": every weight is updated, so the frozen-W
 * shortcut of LoRA no longer applies and the layer also owes  dW = dY^T X):
 *     dW[o, i] = sum_t dY[t, o] X[t, i]        dY [T, d_out] bf16, X [T, d_in] bf16  ->  dW [d_out, d_in] bf16
 * One tcgen05 GEMM over CTA pairs with both operands read token-major as they are (no transposed copies), fp32
 * accumulation over all T tokens, one rounding to bf16.  dW is overwritten; T = 0 gives zeros.  The plan's r plays no
 * role.  Needs the workspace only when the selector split the contraction (cfg.dw_split_k > 1: few output tiles, many
 * tokens); then the splits are summed in a fixed order.  Independent of the other calls. */
int lora_dense_dw(lora_plan_t* plan, const void* dY, const void* X, void* dW, void* stream);

/* Quantised LoRA (Section 4.5, "Quantised LoRA" / Q+LoRA): the same layer with the frozen W held in 4-bit NormalFloat
 * (NF4, Dettmers et al. 2023).  The paper names the data type but no storage layout; this library's is:
 *   - W [d_out, d_in] is cut into blocks of 64 consecutive elements along d_in (d_in % 64 == 0, d_out % 4 == 0);
 *   - W_absmax [d_in / 64, d_out] float32, block-major: W_absmax[b, o] = max |W[o, 64 b .. 64 b + 63]|;
 *   - W_codes [d_out, d_in / 2] uint8: each element's code is the index of the NF4 level nearest to w / absmax
 *     (float32 division; the lower level on an exact tie; an all-zero block gets code 7 = level 0); byte k of a row holds
 *     element 2k in its low nibble and element 2k + 1 in its high nibble;
 *   - the value the GEMMs use is  bf16( float32(level[code]) * absmax )  (one float32 product, one rounding).
 * lora_nf4_quantize builds codes and scales from a bf16 weight on the device (one warp per block);
 * lora_nf4_dequantize expands them to a bf16 matrix W [d_out, d_in] (a streaming kernel, 0.5 + 2 bytes per element).
 * lora_linear_fwd_nf4 / lora_linear_bwd_nf4 compute exactly what lora_linear_fwd / lora_linear_bwd compute with that
 * dequantised weight in place of W; dA and dB do not involve W.  `w_scratch` selects how:
 *   - w_scratch != NULL (caller-owned device memory, d_out * d_in * 2 bytes, 16-byte aligned, contents undefined
 *     afterwards; one buffer can serve every layer of that size): the weight is expanded into it once per call and the
 *     bf16 kernels run on it.  This is the fast form for training batches: each weight element is converted once, not
 *     once per 256-token tile, and the GEMMs keep their shared-memory bandwidth for the tensor cores.
 *   - w_scratch != NULL but SMALLER than the weight, its size announced with lora_plan_set_nf4_scratch_bytes (below):
 *     the weight is expanded band by band (forward: bands of output features, i.e. weight rows; backward: bands of
 *     input features, i.e. weight columns; a band is a whole number of GEMM n-tiles) and the bf16 GEMM runs once per band
 *     on that band's output columns.  Every element is still converted once per call and the results are bit-identical
 *     to the whole-weight form (same tiles, same order of summation); a band of a few MB stays in L2 between its
 *     expansion and the GEMM that reads it.  Costs one expansion launch and one partly filled last wave per band.
 *   - w_scratch == NULL: nothing is materialised; packed codes and scales are staged by TMA and expanded inside the GEMM
 *     kernels, straight into the tensor-core operand tiles.  No extra memory, but the conversion is repeated for every
 *     256-token tile and competes with the tensor cores for shared-memory bandwidth (measured 1.5-2x slower than the
 *     scratch forms from T = 8192 on).  Needs a plan with T > 128, else LORA_ERR_UNSUPPORTED_SHAPE.
 * All three forms give bit-identical weights to the GEMMs.  The workspace must be registered (LORA_ERR_WORKSPACE
 * otherwise; forward needs it in the NULL form and whenever the plan's forward uses it).  All pointers are device
 * pointers, 16-byte aligned. */
/* Size of the buffer behind `w_scratch` in the two Q+LoRA calls of this plan.  lora_plan_nf4_scratch_bytes: `full_bytes` =
 * d_out * d_in * 2 (the whole weight, the default assumption), `min_bytes` = the smallest buffer the banded form accepts
 * (one n-tile of weight rows or columns: max(fwd_block_n * d_in, dx_block_n * d_out) * 2 bytes).
 * lora_plan_set_nf4_scratch_bytes: 0 or anything >= full_bytes selects the whole-weight form; a smaller value the banded
 * form, which needs a plan with T > 128 whose selector did not split the contraction (LORA_ERR_UNSUPPORTED_SHAPE otherwise)
 * and bytes >= min_bytes (LORA_ERR_WORKSPACE otherwise).  The library picks the band height from the size (as many n-tiles
 * as fit, fewer when that leaves fewer idle CTA pairs in the bands' last waves).  Host-side setting, not thread-safe
 * against concurrent calls on the same plan. */
int lora_plan_nf4_scratch_bytes(const lora_plan_t* plan, size_t* min_bytes, size_t* full_bytes);
int lora_plan_set_nf4_scratch_bytes(lora_plan_t* plan, size_t bytes);

int lora_nf4_quantize(const void* W, int64_t d_out, int64_t d_in, void* W_codes, void* W_absmax, void* stream);
int lora_nf4_dequantize(const void* W_codes, const void* W_absmax, int64_t d_out, int64_t d_in, void* W, void* stream);
int lora_linear_fwd_nf4(lora_plan_t* plan, const void* X, const void* W_codes, const void* W_absmax, const void* A,
                        const void* B, float scale, void* Y, void* w_scratch, void* stream);
int lora_linear_bwd_nf4(lora_plan_t* plan, const void* dY, const void* X, const void* W_codes, const void* W_absmax,
                        const void* A, const void* B, float scale, void* dX, void* dA, void* dB, void* w_scratch,
                        void* stream);

/* One training step of the layer with HOST input/output buffers: copies h_X, h_A, h_B, h_dY to the
 * device staging area, runs forward and backward, copies Y, dX, dA, dB back, all on `stream`
 * (asynchronous when the host buffers are pinned).  W is the frozen weight and stays resident on
 * the device.  `staging` is caller-owned device memory of at least lora_step_host_staging_bytes. */
int lora_step_host_staging_bytes(const lora_shape_t* shape, size_t* bytes);
int lora_linear_step_host(lora_plan_t* plan, const void* h_X, const void* W, const void* h_A,
                          const void* h_B, const void* h_dY, float scale, void* h_Y, void* h_dX,
                          void* h_dA, void* h_dB, void* staging, size_t staging_bytes, void* stream);

/* Failure detection.  Every device-side wait (on an mbarrier fed by TMA, by the tensor core or by other warps) gives
 * up after a limit of SM clock ticks; the kernel then records which wait ran out and in which CTA in the plan's status
 * block, lets its copies in flight land, frees its tensor memory and returns, so the context stays usable.
 * lora_last_device_status reports and clears the record.
 *   lora_plan_set_wait_limit   limit for the plan's later launches, in SM clock ticks (default 4e9, about 2 s; 0 restores
 *                              the default; values below 1000 are raised to 1000).  Also settable for new plans through
 *                              the environment variable LORA_DEBUG_WAIT_CAP.
 *   lora_debug_starved_wait    test hook: launches ONE CTA of the adapter-gradient kernel over S [T, C] bf16 (T <= 1024,
 *                              C <= 512, C % 8 == 0) whose second-factor loader issues nothing, so that the MMA warp's
 *                              bounded wait runs out while no copy is outstanding except the few stages of S that
 *                              complete on their own.  `out` ([C, r] fp32) is never written.  Nothing faults or traps; with
 *                              a short limit the launch ends within a millisecond and the next
 *                              lora_last_device_status returns LORA_ERR_DEVICE_TIMEOUT.  */
int lora_plan_set_wait_limit(lora_plan_t* plan, int64_t cycles);
int lora_debug_starved_wait(lora_plan_t* plan, const void* S, int64_t T, int64_t C, void* out, void* stream);

/* Token contraction without any allocation (the paper has no counterpart; this is a library convenience).
 *
 *     out[c, j] = sum_t S[t, c] * Rt[j, t]          S [T, C] bf16, Rt [r, ld_rt] bf16 (ld_rt >= T), out [C, r] fp32
 *
 * This is the kernel behind dB = scale dY^T (X A^T) with S = dY and Rt = the caller's bf16 copy of
 * scale (X A^T)^T, usable on its own.  It is meant for callers that must not allocate device memory when
 * they call in: code running under a memory pool that forbids cudaMalloc after start-up, real-time or
 * inference loops where an allocation would stall the device, and hosts that hand this library a fixed
 * memory budget.  No plan is needed (creating one allocates a status block).  Nothing in this call
 * allocates or frees: the only global scratch the kernel needs - its status block, where a device-side wait that ran out
 * is recorded - lives in one static device array of lora_grad_contract_noalloc_max_scratch() bytes (4 KiB) that every
 * GPU loading the library holds until the process exits.  (The sums over token chunks meet on chip, in the distributed
 * shared memory of a thread-block cluster, so there are no partial sums in global memory to make room for.)
 *   - Limits: C % 8 == 0, r in {8,...,64}, ld_rt % 8 == 0, 1 <= T <= 2^30, C <= 2^24; anything beyond is rejected with
 *     LORA_ERR_UNSUPPORTED_SHAPE (LORA_ERR_INVALID_ARG for null pointers or ld_rt < T) before anything is launched.
 *   - The first call on a device looks up the array's device address, raises the kernel's shared-memory
 *     limit and asks how many clusters fit the device; make that first call before any stream capture.  The current
 *     device is used.
 *   - All calls share the one array and it keeps the last call's contents; the call clears it on `stream` first.
 *     Two calls whose kernels overlap on the GPU (different streams, or different host threads) race on it: serialise them.
 *   - A bounded device wait that ran out leaves `out` incomplete while the call itself has long returned LORA_OK:
 *     lora_grad_contract_noalloc_status synchronises `stream`, reads the status word of the current device's array
 *     (a 4-byte copy, no allocation) and sets *code to LORA_OK or LORA_ERR_DEVICE_TIMEOUT. */
int lora_grad_contract_noalloc(const void* S, const void* Rt, int64_t T, int64_t C, int64_t r, int64_t ld_rt,
                               void* out, void* stream);
int lora_grad_contract_noalloc_status(void* stream, int* code);
int64_t lora_grad_contract_noalloc_max_scratch(void);

/* Synchronise `stream`, then report whether any kernel of this plan gave up on a bounded wait.
 * *code is LORA_OK or LORA_ERR_DEVICE_TIMEOUT; msg (may be NULL) receives a short description.
 * The status word is cleared. */
int lora_last_device_status(lora_plan_t* plan, void* stream, int* code, char* msg, size_t n);

/* SM clock of the last CTA-pair GEMM launch of this plan (forward or dX, whichever ran last), measured inside the kernel:
 * one thread reads the nanosecond wall timer and the SM cycle counter when its CTA starts working and when it leaves; their
 * ratio is the frequency the launch really ran at (external polling of the driver's clock readout is too slow to see
 * millisecond launches under a power cap).  Synchronises `stream`.  *sm_mhz = 0 when no such launch ran yet. */
int lora_plan_last_gemm_clock(lora_plan_t* plan, void* stream, double* sm_mhz, double* busy_us);

/* Static string for a status code. */
const char* lora_strerror(int code);

/* Number of kernels the library has launched in this process (all plans). */
int64_t lora_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* LORA_LINEAR_H_ */
