// Internal launcher interface between the C ABI (api.cu) and the kernels.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <utility>

namespace lora {

// Launch with programmatic stream serialization: the grid may begin (prologue only, see pdl_wait in the kernels)
// before the preceding kernel of the stream has drained.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Default limit of every device-side spin, in SM clock ticks (~2 s at 2 GHz)
constexpr long long kWaitLimitCycles = 4000000000LL;

// ---- dense GEMM + fused rank-r adapter (forward Y, backward dX) -------------------------------
constexpr int kBlockM = 128;          // token rows per tile (one TMEM lane per row)
constexpr int kBlockK = 64;           // contraction elements per stage (one 128-byte swizzle row)
constexpr int kStageABytes = kBlockM * 128;
constexpr int kStageBBytes = 256 * 128;
constexpr int kStageBytes = kStageABytes + kStageBBytes;
constexpr int kStagingBytes = 128 * 128;   // one 128 x 64 bf16 output chunk / the bf16 rank-r operand
constexpr int kGemmThreads = 192;          // warp 0 TMA, warp 1 MMA + TMEM, warps 2..5 epilogue
constexpr int kMaxStages = 8;
constexpr int kGemmBarriers = 2 * kMaxStages + 8;

struct GemmParams {
  int M, N, K;            // output rows (tokens), output columns, contraction length
  int r_pad;              // rank rounded up to a multiple of 16
  int block_n;            // output columns per tile: 64, 128 or 192
  int tiles_m, tiles_n, num_tiles, kblocks;
  int group_m;            // m-tiles per rasterisation band
  int stages;             // ring depth
  int prefetch_dist;      // CTA-pair kernel: k-blocks by which L2 prefetches run ahead of the ring (0 = off)
  int tail_delay;         // main-loop k-blocks of the next tile issued before the previous tile's rank-r MMA
  float scale;
  __nv_bfloat16* rt_out;  // backward only: scale * (dY B)^T as bf16 [r_pad][ld_rt]; nullptr otherwise
  int ld_rt;
  unsigned* status;       // device status word
  long long wait_limit;   // SM clock ticks after which a spin gives up and reports through `status`
  int split_k;            // K-extended pair kernel: k-splits per tile (1 = none) and main k-blocks per split
  int kb_per_split;
  float* part;            // fp32 partial tiles [split_k][M][N] when split_k > 1
  __nv_bfloat16* out;     // CTA-pair kernel only: output base and row pitch (elements) for the ragged last chunk
  int ld_out;
  // K-extended CTA-pair kernel, grouped projections (several projections share the activations; see lora_linear_fwd_grouped):
  int tail_parts;         // rank-r k-blocks per tile (>= 1; the dX GEMM of G groups adds G of them, rows part x r_pad)
  int n_groups;           // forward: output-column groups (<= 1: ungrouped); a tile's rank-r k-block uses the rows
  int group_end[4];       //   group x r_pad of s (X A^T)^T, group = first g with n0 < group_end[g]
};

size_t gemm_smem_bytes(int stages);

// ---- CTA-pair (cta_group::2) variant: 256-row tiles, block_n a multiple of 16 with block_n + r_pad <= 256 ----
constexpr int kPairBlockM = 256;
constexpr int kPairThreads = 288;           // warps 0..3 TMA producers, warp 4 MMA + TMEM, warps 5..8 epilogue
constexpr int kPairStageBytesFwd = 32768;   // 128 x 64 activations + 128 x 64 weight/adapter rows per CTA
// NF4 weight (K-extended forms only): eight more warps dequantise; packed codes + block scales travel through a ring of
// kNf4CodeSlots slots of 4096 code bytes + 128 float scales
constexpr int kNf4DequantThreads = 256;
constexpr int kNf4Groups = 4;               // ring items are dealt round-robin to groups of dequantising warps
constexpr int kNf4WarpsPerGroup = kNf4DequantThreads / 32 / kNf4Groups;
constexpr int kPairThreadsNf4 = kPairThreads + kNf4DequantThreads;
constexpr int kNf4CodeSlots = 6;
constexpr int kNf4CodeSlotBytes = 4096 + 512;
constexpr int kNf4Block = 64;               // elements per quantisation block (= kBlockK)
size_t gemm_pair_smem_bytes(int stages, bool nf4 = false);
cudaError_t gemm_pair_configure();
// out = bf16(sum of the split_k fp32 partial matrices), fixed order (M x N must be a multiple of 8 elements)
cudaError_t launch_splitk_reduce(const float* part, __nv_bfloat16* out, long long n_elems, int splits, cudaStream_t stream);
// forward: tmW0 = W box 64 x half rows (leader CTA), tmW1 = W box 64 x (block_n - half) rows (peer CTA),
// half = (block_n + r_pad) / 2; tmA box 64 x r_pad; tmB box 64 x block_n/2 rows
cudaError_t launch_gemm_pair_fwd(const CUtensorMap& tmX, const CUtensorMap& tmW0, const CUtensorMap& tmW1,
                                 const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmY,
                                 const GemmParams& p, int ctas, cudaStream_t stream);
// K-extended forward (adapter's X A^T computed beforehand): tmW box 64(k) x block_n/2 rows; tmPt = s (X A^T)^T [r_pad, T]
// box 64(t) x r_pad; tmB box 64(r) x block_n/2 rows
cudaError_t launch_gemm_pair_fwd_ext(const CUtensorMap& tmX, const CUtensorMap& tmW, const CUtensorMap& tmPt,
                                     const CUtensorMap& tmB, const CUtensorMap& tmY, const GemmParams& p, int ctas,
                                     cudaStream_t stream);
// backward: tmW box 64(n) x 64(k); tmQt = s (dY B)^T [r_pad, T] box 64(t) x r_pad; tmA box 64(n) x r_pad
cudaError_t launch_gemm_pair_dx(const CUtensorMap& tmdY, const CUtensorMap& tmW, const CUtensorMap& tmQt,
                                const CUtensorMap& tmA, const CUtensorMap& tmdX, const GemmParams& p, int ctas,
                                cudaStream_t stream);

// NF4 frozen weight: tmCodes = packed codes [d_out, d_in/2] uint8, no swizzle, box 32 B x 128 rows (forward) or
// 64 B x 64 rows (backward); tmAbsmax = block scales [d_in/64, d_out] float, box 128 x 1 (forward) or 64 x 2 (backward);
// the other maps as in the K-extended bf16 launchers.  Forward block_n any multiple of 16, backward block_n = 256.
cudaError_t launch_gemm_pair_fwd_nf4(const CUtensorMap& tmX, const CUtensorMap& tmCodes, const CUtensorMap& tmAbsmax,
                                     const CUtensorMap& tmPt, const CUtensorMap& tmB, const CUtensorMap& tmY,
                                     const GemmParams& p, int ctas, cudaStream_t stream);
cudaError_t launch_gemm_pair_dx_nf4(const CUtensorMap& tmdY, const CUtensorMap& tmCodes, const CUtensorMap& tmAbsmax,
                                    const CUtensorMap& tmQt, const CUtensorMap& tmA, const CUtensorMap& tmdX,
                                    const GemmParams& p, int ctas, cudaStream_t stream);
// W [d_out, d_in] bf16 -> NF4 codes [d_out, d_in/2] + block scales [d_in/64, d_out] (nf4_quant.cu)
cudaError_t launch_nf4_quantize(const __nv_bfloat16* W, long long d_out, long long d_in, uint8_t* codes, float* absmax,
                                cudaStream_t stream);

// NF4 codes + block scales -> bf16 weight [d_out, d_in], every element bf16(level * absmax) (nf4_quant.cu)
cudaError_t launch_nf4_dequantize(const uint8_t* codes, const float* absmax, long long d_out, long long d_in, __nv_bfloat16* W,
                                  int num_sms, cudaStream_t stream);
// the same for the window rows [o0, o0 + n_rows) x columns [c0, c0 + n_cols) of the weight (c0, n_cols, ld_w multiples of 8:
// a thread expands one 32-bit code word into 16 bytes), written to W with a row pitch of ld_w elements
cudaError_t launch_nf4_dequantize_window(const uint8_t* codes, const float* absmax, long long d_out, long long d_in, long long o0,
                                         long long n_rows, long long c0, long long n_cols, __nv_bfloat16* W, long long ld_w,
                                         int num_sms, cudaStream_t stream);

// dense weight gradient dW[d_out, d_in] = dY^T X (p.r_pad = 0: no rank-r k-block): tmdYt = dY [T, d_out] box 64(o) x 64(t),
// tmX = X [T, d_in] box 64(i) x 64(t), tmdW box 64 x 128; p.M = d_out, p.N = d_in, p.K = T
cudaError_t launch_gemm_pair_dw(const CUtensorMap& tmdYt, const CUtensorMap& tmX, const CUtensorMap& tmdW, const GemmParams& p,
                                int ctas, cudaStream_t stream);

// Y / dX = act * Wop + scale * (act * sideop) * tailop, see gemm_lora.cu
cudaError_t launch_gemm_fwd(const CUtensorMap& tmX, const CUtensorMap& tmW, const CUtensorMap& tmA,
                            const CUtensorMap& tmB, const CUtensorMap& tmY, const GemmParams& p, int ctas,
                            cudaStream_t stream);
cudaError_t launch_gemm_dx(const CUtensorMap& tmdY, const CUtensorMap& tmW, const CUtensorMap& tmB,
                           const CUtensorMap& tmA, const CUtensorMap& tmdX, const GemmParams& p, int ctas,
                           cudaStream_t stream);
cudaError_t gemm_configure();   // opt in to the large dynamic shared memory (once per device)

// ---- adapter gradients and skinny side products: tall-skinny contractions over one stream of tokens --------
constexpr int kGradProducerWarps = 4;      // warps 0..3: TMA producers of the streamed tiles (ring items round-robin)
constexpr int kGradEpiGroups = 2;          // two groups of four epilogue warps; the per-slab work alternates between them
constexpr int kGradThreads = 32 * (kGradProducerWarps + 2 + 4 * kGradEpiGroups);   // + MMA warp + second-factor loader
constexpr int kGradSlab = 128;             // tokens per slab
constexpr int kGradStageBytes = 2 * kBlockM * 128;   // 128 tokens x 128 features, bf16
constexpr int kGradMaxStages = 6;
constexpr int kGradMaxRtBufs = 4;          // ring of second-factor slabs (a gradient CTA with one block needs one per tile)
constexpr int kGradPBufs = 4;              // TMEM buffers of the per-slab side product (r_pad columns each)
constexpr int kGradMaxCluster = 16;        // token chunks of one feature chunk form a thread-block cluster of this size at most

struct GradParams {
  int T, C;               // tokens, features of the streamed matrix (d_in for dA, d_out for dB)
  int r, r_pad;
  int feat_chunk;         // features per CTA (multiple of 128)
  int n_feat_chunks;      // grid x
  int n_token_chunks;     // grid y = cluster size along y when do_out (the cluster sums the gradient over its token chunks)
  int n_slabs;
  int stages;
  int rt_bufs;            // depth of the second-factor ring (1 .. kGradMaxRtBufs)
  int rt_in_stage;        // 1: the second factor's slab travels in each tile's own stage (one-block gradient CTAs)
  int tmem_cols;          // TMEM columns to allocate (power of two >= 32)
  int with_p;             // 1: also accumulate the side product S * side^T for each slab (X A^T, or dY B)
  int side_mn;            // side operand: 0 = A [r, C] (K-major rows), 1 = B [C, r] (MN-major, natural layout)
  int do_out;             // 0: side product only (no second factor, no gradient)
  int out_is_da;          // 1: out[j * C + c] (dA), 0: out[c * r + j] (dB)
  int accumulate;         // 1: out += result (gradient accumulation over micro-batches), 0: out = result
  float scale;
  float* out;             // final fp32 gradient
  float* p_part;          // [n_feat_chunks][r_pad][ld_t] partial X A^T (with_p and more than one feature chunk)
  int* side_count;        // [n_slabs] arrival counters of the side-product partials; zero before and after every launch
  __nv_bfloat16* pt_out;  // [r_pad][ld_t]: scale * (X A^T)^T as bf16 (with_p)
  int ld_t;
  unsigned* status;
  long long wait_limit;   // SM clock ticks after which a spin gives up and reports through `status`
  int debug_no_second_factor;   // test hook: the second-factor loader issues nothing, so the MMA warp's wait runs out
};

// What the grid rule chose for one streaming launch
struct GradGrid {
  int feat_chunk, n_feat, n_tok, stages, tmem_cols;
};
// Grid of a launch that computes the gradient of one streamed matrix with C features (with or without the side product),
// or of two matrices with C and C2 features side by side (C2 = 0: one job): feature chunk width and cluster size
// (= token chunks) with the lowest modelled time among those that fit TMEM (feat_chunk / 128 x r_pad + side buffers <= 512
// columns) and are resident at once (caps[cs] = CTAs resident at once in clusters of cs CTAs, cs = 1 .. kGradMaxCluster).
// n_feat counts the feature chunks of both jobs.
GradGrid grad_pick_grid(long long T, long long C, long long C2, int r_pad, bool with_p, bool side_mn, const int* caps);
// the same for n_jobs streamed matrices with C[j] features side by side (r_pad: the largest of the jobs)
GradGrid grad_pick_grid_jobs(long long T, const long long* C, int n_jobs, int r_pad, bool with_p, bool side_mn, const int* caps);
// caps[0 .. kGradMaxCluster] estimated from the SM count alone (host-only selector calls) / asked from the current device
void grad_default_caps(int num_sms, int* caps);
void grad_device_caps(int num_sms, int* caps);
// TMEM columns a launch allocates: gradient sums + side-product buffers, rounded up to a power of two >= 32
int grad_tmem_cols(int feat_chunk, int r_pad, bool do_out, bool with_p);



// One launch of the streaming kernel: up to kGradMaxJobs jobs side by side (CTAs with blockIdx.x in [x_end[j-1], x_end[j])
// run job j)
constexpr int kGradMaxJobs = 6;
struct GradLaunch {
  GradParams job[kGradMaxJobs];
  int x_end[kGradMaxJobs];
  int n_jobs;
};
struct GradMaps {
  CUtensorMap m[3 * kGradMaxJobs];       // per job: streamed matrix, second factor, side operand
};
// what the host passes per job
struct GradJobDesc {
  CUtensorMap tmS, tmR, tmSide;
  GradParams p;
};

size_t grad_smem_bytes(const GradParams& p);
// ring geometry of a job from its other fields (do_out, with_p, side_mn, r_pad, feat_chunk): sets stages, rt_bufs, rt_in_stage
void grad_set_ring(GradParams* p);
// opt in to the large dynamic shared memory and to clusters of more than 8 CTAs (once per device)
cudaError_t grad_configure();
// Largest grid (in CTAs) of `cluster`-CTA clusters along y that is resident at once on the current device, for the given
// launch shape; 0 when the query fails.
int grad_max_resident_ctas(int cluster, size_t smem_bytes);
// tmS: streamed matrix [T, C] box [64 features, 128 tokens]; tmR: [r_pad, T] box [64 tokens, r_pad];
// tmA: side operand (only read when with_p).  ONE launch: the gradient is summed over the token chunks inside the cluster
// (distributed shared memory, rank order), the side product over the feature chunks by the last CTA to arrive (chunk order).
cudaError_t launch_grad(const CUtensorMap& tmS, const CUtensorMap& tmR, const CUtensorMap& tmA,
                        const GradParams& p, cudaStream_t stream);
// Several jobs in one launch.  All jobs compute a gradient with the same cluster size, or all compute only a side product.
cudaError_t launch_grad_jobs(const GradJobDesc* jobs, int n_jobs, cudaStream_t stream);

}  // namespace lora
