// Adapter gradients of the LoRA layer (Section 3.2.2, LoRA): tall-skinny contractions over the tokens.
//
//   dA = s (dY B)^T X      streams X  [T, d_in]  once, second factor Qt = s (dY B)^T  [r_pad, T] (bf16)
//   dB = s dY^T (X A^T)    streams dY [T, d_out] once, second factor Pt = s (X A^T)^T [r_pad, T] (bf16)
//
// Both are out[c, j] = sum_t S[t, c] * Rt[j, t]: the streamed matrix S is the MN-major A operand of a
// tcgen05 MMA (M = 128 features, N = r_pad, K = tokens) read from the very 128-byte-swizzled tiles TMA
// delivers, so the token reduction runs on the tensor cores while the kernel stays bound by the HBM
// stream.  The dA kernel additionally recomputes X A^T for the slab it holds (same tiles, this time as the
// K-major operand with M = 128 tokens), because the backward pass is not given the forward's X A^T.
//
// Grid: (feature chunks, token chunks), at most one CTA per SM.  A CTA keeps feat_chunk x r_pad fp32 sums in
// TMEM over all of its token slabs.  Cross-CTA sums (over token chunks for the gradient, over feature chunks
// for X A^T) are written as fp32 partials and added in a fixed order by lora_grad_finalize_kernel, so the
// result is bitwise reproducible and no CTA ever waits for another.
//
// The side product has two operand forms: A [r, C] (K-major rows, for X A^T) or B [C, r] (MN-major, its natural
// layout, for dY B); with do_out = 0 the kernel computes only the side product (the Q = dY B pre-pass of backward).
//
// Warps: 0, 1 TMA producers of the streamed tiles (even / odd ring items: one warp's copies sustain only
// ~30 B/clk), 2 MMA issuer + TMEM, 3 loader of the second factor, 4..7 epilogue.
#include "kernels.h"
#include "sm100_ptx.cuh"

#include <mutex>

#include "../../include/lora_linear.h"

namespace lora {

namespace {

constexpr int kGradBarriers = 2 * kGradMaxStages + 10;

__global__ void __launch_bounds__(kGradThreads, 1)
lora_grad_kernel(const __grid_constant__ CUtensorMap tm_s,   // streamed matrix [T, C], box 64(c) x 128(t)
                 const __grid_constant__ CUtensorMap tm_r,   // second factor [r_pad, T], box 64(t) x r_pad
                 const __grid_constant__ CUtensorMap tm_a,   // side operand (with_p): A [r, C] box 64(c) x r_pad, or
                                                             // B [C, r] box 64(r, zero-filled) x 64(c) when side_mn
                 const GradParams p) {
  pdl_launch_dependents();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int NB = p.feat_chunk >> 7;                 // 128-feature accumulator blocks
  const int rt_box = p.r_pad * 128;                 // bytes of one 64-wide box with r_pad rows
  const int side_box = p.side_mn ? 8192 : rt_box;   // bytes of the side operand for 64 features
  const int stage_bytes = kGradStageBytes + (p.with_p ? 2 * side_box : 0);   // S tile (+ the matching side operand)
  const uint32_t ring = smem_u32(smem);
  const uint32_t rt_base = ring + p.stages * stage_bytes;               // 2 buffers x 2 boxes of the second factor
  uint8_t* tail = smem + p.stages * stage_bytes + 4 * rt_box;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tail);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kGradMaxStages + s); };
  auto rt_full = [&](int b) { return bar0 + 8u * (2 * kGradMaxStages + b); };
  auto rt_empty = [&](int b) { return bar0 + 8u * (2 * kGradMaxStages + 2 + b); };
  auto p_full = [&](int b) { return bar0 + 8u * (2 * kGradMaxStages + 4 + b); };
  auto p_empty = [&](int b) { return bar0 + 8u * (2 * kGradMaxStages + 6 + b); };
  const uint32_t out_full = bar0 + 8u * (2 * kGradMaxStages + 8);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kGradBarriers);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int fc = blockIdx.x, tc = blockIdx.y;
  const int c0 = fc * p.feat_chunk;
  const int s_begin = static_cast<int>(static_cast<long long>(tc) * p.n_slabs / p.n_token_chunks);
  const int s_end = static_cast<int>(static_cast<long long>(tc + 1) * p.n_slabs / p.n_token_chunks);
  const int S = p.stages;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(rt_full(b), 1);
      mbar_init(rt_empty(b), 1);
      mbar_init(p_full(b), 1);
      mbar_init(p_empty(b), 128);
    }
    mbar_init(out_full, 1);
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tm_s);
    tma_prefetch_desc(&tm_r);
    if (p.with_p) tma_prefetch_desc(&tm_a);
  }
  if (warp == 2) {
    tmem_alloc(smem_u32(tmem_slot), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();                   // global memory of earlier kernels is visible from here on
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_p = tmem_base + (p.do_out ? NB * p.r_pad : 0);     // two r_pad-column buffers for the side product

  if (warp < 2) {
    // ================================ TMA producers: streamed tiles, even / odd ring items ================================
    int slot = 0, phase = 0, odd = 0;
    bool ok = true;
    for (int s = s_begin; s < s_end && ok; ++s) {
      const int t0 = s * kGradSlab;
      for (int nb = 0; nb < NB && ok; ++nb) {
        if (odd == warp) {
          ok = warp_wait(empty_bar(slot), phase ^ 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_EMPTY, false, 20);
          if (ok && elect_one()) {
            const uint32_t dst = ring + slot * stage_bytes, fb = full_bar(slot);
            const int cc = c0 + nb * 128;
            mbar_arrive_expect_tx(fb, stage_bytes);
            tma_load_2d(dst, &tm_s, fb, cc, t0);
            tma_load_2d(dst + 16384, &tm_s, fb, cc + 64, t0);
            if (p.with_p && !p.side_mn) {
              tma_load_2d(dst + 32768, &tm_a, fb, cc, 0);
              tma_load_2d(dst + 32768 + side_box, &tm_a, fb, cc + 64, 0);
            } else if (p.with_p) {
              tma_load_2d(dst + 32768, &tm_a, fb, 0, cc);
              tma_load_2d(dst + 32768 + side_box, &tm_a, fb, 0, cc + 64);
            }
          }
          __syncwarp();
        }
        if (++slot == S) { slot = 0; phase ^= 1; }
        odd ^= 1;
      }
    }
  } else if (warp == 3) {
    // ================================ loader of the second factor (one 128-token slab at a time) ================================
    bool ok = true;
    int rb = 0, rphase = 0;
    for (int s = s_begin; s < s_end && ok && p.do_out && !p.debug_no_second_factor; ++s) {
      ok = warp_wait(rt_empty(rb), rphase ^ 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_EMPTY, false, 20);
      if (ok && elect_one()) {
        const int t0 = s * kGradSlab;
        mbar_arrive_expect_tx(rt_full(rb), 2 * rt_box);
        tma_load_2d(rt_base + (2 * rb) * rt_box, &tm_r, rt_full(rb), t0, 0);
        tma_load_2d(rt_base + (2 * rb + 1) * rt_box, &tm_r, rt_full(rb), t0 + 64, 0);
      }
      __syncwarp();
      if (++rb == 2) { rb = 0; rphase ^= 1; }
    }
  } else if (warp == 2) {
    // ================================ MMA issuer ================================
    const uint32_t idesc_out = mma_idesc_bf16(128, p.r_pad, true, false);   // A operand = S tile, MN-major
    const uint32_t idesc_p = mma_idesc_bf16(128, p.r_pad, false, p.side_mn != 0);   // A operand = S tile, K-major
    const uint64_t a_mn0 = smem_desc_sw128(ring, 16384, 1024);              // S tile as [features x tokens]
    const uint64_t a_k0 = smem_desc_sw128(ring, 16, 1024);                  // S tile as [tokens x features]
    const uint64_t w_k0 = smem_desc_sw128(ring + 32768, 16, 1024);          // side operand of the stage
    const uint32_t sbox = static_cast<uint32_t>(side_box) >> 4;
    const uint32_t sstep = p.side_mn ? 128u : 2u;                           // descriptor step per 16 features
    const uint64_t r_k0 = smem_desc_sw128(rt_base, 16, 1024);               // second factor
    bool ok = true;
    int slot = 0, phase = 0, rb = 0, rphase = 0;
    for (int s = s_begin; s < s_end && ok; ++s) {
      if (p.do_out) ok = warp_wait(rt_full(rb), rphase, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_FULL, false, 0);
      if (ok && p.with_p) ok = warp_wait(p_empty(rb), rphase ^ 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_ACC_EMPTY, false, 0);
      for (int nb = 0; nb < NB && ok; ++nb) {
        ok = warp_wait(full_bar(slot), phase, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_FULL, false, 0);
        if (!ok) break;
        tc_fence_after();
        if (elect_one()) {
          const uint32_t so = static_cast<uint32_t>(slot * stage_bytes) >> 4;
          const uint32_t ro = static_cast<uint32_t>(2 * rb * rt_box) >> 4;
          const uint32_t rbox = static_cast<uint32_t>(rt_box) >> 4;
          if (p.do_out) {
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)   // 128 tokens = 8 x K16; second factor: box ks/4, 32 B per k-step
              mma_bf16_ss(tmem_base + nb * p.r_pad, a_mn0 + so + ks * 128, r_k0 + ro + (ks >> 2) * rbox + (ks & 3) * 2,
                          idesc_out, (s != s_begin || ks != 0) ? 1u : 0u);
          }
          if (p.with_p) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)   // 128 features = 2 boxes x 4 x K16
              mma_bf16_ss(tmem_p + rb * p.r_pad, a_k0 + so + (kk >> 2) * 1024 + (kk & 3) * 2,
                          w_k0 + so + (kk >> 2) * sbox + (kk & 3) * sstep, idesc_p, (nb != 0 || kk != 0) ? 1u : 0u);
          }
          mma_commit(empty_bar(slot));
          if (nb == NB - 1) {
            if (p.do_out) mma_commit(rt_empty(rb));
            if (p.with_p) mma_commit(p_full(rb));
          }
        }
        __syncwarp();
        if (++slot == S) { slot = 0; phase ^= 1; }
      }
      if (++rb == 2) { rb = 0; rphase ^= 1; }
    }
    if (ok && p.do_out && elect_one()) mma_commit(out_full);
    __syncwarp();
  } else {
    // ================================ epilogue (warps 4..7, 128 threads) ================================
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
    bool alive = true;
    if (p.with_p) {
      // ---- X A^T of each slab, partial over this CTA's features -> p_part[fc][j][t] ----
      int pb = 0, pphase = 0;
      for (int s = s_begin; s < s_end; ++s) {
        const int t = s * kGradSlab + row;
        bool ok = warp_wait(p_full(pb), pphase, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_SIDE, false, 32);
        if (named_bar_or(1, 128, !ok)) { alive = false; break; }
        tc_fence_after();
        for (int c16 = 0; c16 < p.r_pad / 16; ++c16) {
          uint32_t v[16];
          tmem_ld16(tmem_p + lane_addr + pb * p.r_pad + c16 * 16, v);
          tmem_ld_wait();
          if (t < p.T && !p.direct) {
#pragma unroll
            for (int q = 0; q < 16; ++q)
              p.p_part[(static_cast<size_t>(fc) * p.r_pad + c16 * 16 + q) * p.ld_t + t] = __uint_as_float(v[q]);
          } else if (t < p.T) {
            // this CTA holds every feature: the side product is complete, write bf16(scale * .) straight to its place
            unsigned short* pt = reinterpret_cast<unsigned short*>(p.pt_out);
#pragma unroll
            for (int q = 0; q < 16; ++q)
              pt[static_cast<size_t>(c16 * 16 + q) * p.ld_t + t] =
                  static_cast<unsigned short>(pack_bf16x2(__uint_as_float(v[q]) * p.scale, 0.f) & 0xFFFFu);
          }
        }
        tc_fence_before();
        mbar_arrive(p_empty(pb));
        if (++pb == 2) { pb = 0; pphase ^= 1; }
      }
    }
    if (alive && p.do_out) {
      bool ok = warp_wait(out_full, 0, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_ACC, false, 32);
      if (!named_bar_or(1, 128, !ok)) {
        tc_fence_after();
        // ---- this CTA's sums over its token chunk -> out_part[tc][j][c] ----
        for (int nb = 0; nb < NB; ++nb) {
          const int c = c0 + nb * 128 + row;
          for (int c16 = 0; c16 < p.r_pad / 16; ++c16) {
            uint32_t v[16];
            tmem_ld16(tmem_base + lane_addr + nb * p.r_pad + c16 * 16, v);
            tmem_ld_wait();
            if (c < p.C && !p.direct) {
#pragma unroll
              for (int q = 0; q < 16; ++q)
                p.out_part[(static_cast<size_t>(tc) * p.r_pad + c16 * 16 + q) * p.c_pad + c] = __uint_as_float(v[q]);
            } else if (c < p.C) {
              // the only token chunk: the sums are final, write them where the finalize kernel would have
#pragma unroll
              for (int q = 0; q < 16; ++q) {
                const int j = c16 * 16 + q;
                if (j < p.r) {
                  float* dst = p.out_is_da ? p.out + static_cast<size_t>(j) * p.C + c : p.out + static_cast<size_t>(c) * p.r + j;
                  *dst = p.accumulate ? *dst + __uint_as_float(v[q]) : __uint_as_float(v[q]);
                }
              }
            }
          }
        }
      }
    }
  }

  // ================================ teardown ================================
  tc_fence_before();
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0) {
    const long long t0 = clock64();          // bounded grace period for copies still in flight
    while (clock64() - t0 < 2000000LL) {
    }
  }
  __syncthreads();
  if (warp == 2) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// Sum of `n` floats spaced `stride` apart, added in index order; loads are issued eight at a time so that their
// latencies overlap (the additions stay sequential, so the result does not depend on the batching).  Larger batches
// were measured slower (32 at a time: 80 registers, +4 us on the dA finalize).
__device__ __forceinline__ float ordered_sum(const float* p, int n, size_t stride) {
  float acc = 0.f;
  int k = 0;
  for (; k + 8 <= n; k += 8) {
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __ldcg(p + static_cast<size_t>(k + i) * stride);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc += v[i];
  }
  for (; k < n; ++k) acc += __ldcg(p + static_cast<size_t>(k) * stride);
  return acc;
}

// Fixed-order sums of the partials:  out = sum over token chunks of out_part ;  Pt = bf16(scale * sum over feature
// chunks of p_part).  One thread per output element, consecutive threads on consecutive addresses.
__global__ void __launch_bounds__(256) lora_grad_finalize_kernel(const GradParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const long long n_out = p.do_out ? static_cast<long long>(p.r) * p.C : 0;
  const long long n_pt = p.with_p ? static_cast<long long>(p.r_pad) * p.T : 0;
  const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx < n_out) {
    const int j = static_cast<int>(idx / p.C), c = static_cast<int>(idx - static_cast<long long>(j) * p.C);
    const float acc = ordered_sum(p.out_part + static_cast<size_t>(j) * p.c_pad + c, p.n_token_chunks,
                                  static_cast<size_t>(p.r_pad) * p.c_pad);
    float* dst = p.out_is_da ? p.out + static_cast<size_t>(j) * p.C + c : p.out + static_cast<size_t>(c) * p.r + j;
    *dst = p.accumulate ? *dst + acc : acc;      // gradient accumulation: old value + (partials in fixed order)
  } else if (idx < n_out + n_pt) {
    const long long i2 = idx - n_out;
    const int j = static_cast<int>(i2 / p.T), t = static_cast<int>(i2 - static_cast<long long>(j) * p.T);
    const float acc = ordered_sum(p.p_part + static_cast<size_t>(j) * p.ld_t + t, p.n_feat_chunks,
                                  static_cast<size_t>(p.r_pad) * p.ld_t);
    reinterpret_cast<unsigned short*>(p.pt_out)[static_cast<size_t>(j) * p.ld_t + t] =
        static_cast<unsigned short>(pack_bf16x2(acc * p.scale, 0.f) & 0xFFFFu);
  }
}

}  // namespace

size_t grad_smem_bytes(const GradParams& p) {
  const size_t stage = kGradStageBytes + (p.with_p ? 2 * (p.side_mn ? size_t(8192) : static_cast<size_t>(p.r_pad) * 128) : 0);
  return static_cast<size_t>(p.stages) * stage + 4 * static_cast<size_t>(p.r_pad) * 128 + kGradBarriers * 8 + 16 + 1024;
}

cudaError_t grad_configure() {
  return cudaFuncSetAttribute(lora_grad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
}

bool grad_is_direct(const GradParams& p) {
  return (!p.do_out || p.n_token_chunks == 1) && (!p.with_p || p.n_feat_chunks == 1);
}

cudaError_t launch_grad(const CUtensorMap& tmS, const CUtensorMap& tmR, const CUtensorMap& tmA, const GradParams& p_in,
                        cudaStream_t stream) {
  GradParams p = p_in;
  // No cross-CTA sum left (one token chunk for the gradient, one feature chunk for the side product): the streaming
  // kernel writes the results itself and the finalize launch is dropped.  Only tiny problems have such grids.
  p.direct = grad_is_direct(p) ? 1 : 0;
  dim3 grid(p.n_feat_chunks, p.n_token_chunks);
  cudaError_t e = launch_pdl(lora_grad_kernel, grid, dim3(kGradThreads), grad_smem_bytes(p), stream, tmS, tmR, tmA, p);
  if (e != cudaSuccess || p.direct) return e;
  const long long n = (p.do_out ? static_cast<long long>(p.r) * p.C : 0) + (p.with_p ? static_cast<long long>(p.r_pad) * p.T : 0);
  return launch_pdl(lora_grad_finalize_kernel, dim3(static_cast<unsigned>((n + 255) / 256)), dim3(256), 0, stream, p);
}

// ================================================================================================
// No-allocation variant of the dB-style contraction: scratch lives in a static device array
// ================================================================================================
namespace {

// Scratch held by every GPU that loads this library, until the process exits: one status block and the
// per-token-chunk partial sums of the contraction kernel.
constexpr size_t kNoAllocScratchBytes = 8u << 20;
constexpr size_t kNoAllocHeaderBytes = 4096;     // [0,256) status words, rest reserved
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

struct NoAllocDevice {
  bool ready = false;
  unsigned char* scratch = nullptr;   // device address of g_noalloc_scratch on this device
  int num_sms = 0;
};
constexpr int kNoAllocMaxDevices = 64;
NoAllocDevice g_noalloc_dev[kNoAllocMaxDevices];
std::mutex g_noalloc_mutex;

typedef CUresult (*NoAllocEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool noalloc_tmap(CUtensorMap* m, const void* ptr, uint64_t inner, uint64_t outer, uint64_t pitch_elems,
                  uint32_t box_inner, uint32_t box_outer) {
  static NoAllocEncodeFn fn = []() -> NoAllocEncodeFn {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess) return nullptr;
    return q == cudaDriverEntryPointSuccess ? reinterpret_cast<NoAllocEncodeFn>(f) : nullptr;
  }();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {inner, outer};
  const cuuint64_t strides[1] = {pitch_elems * 2};
  const cuuint32_t box[2] = {box_inner, box_outer};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace
}  // namespace lora

extern "C" int lora_grad_contract_noalloc(const void* S, const void* Rt, int64_t T, int64_t C, int64_t r,
                                          int64_t ld_rt, void* out, void* stream) {
  using namespace lora;
  if (!S || !Rt || !out) return LORA_ERR_INVALID_ARG;
  if (T <= 0 || C <= 0 || r <= 0 || ld_rt < T) return LORA_ERR_INVALID_ARG;
  if (C % 8 != 0 || r % 8 != 0 || r > 64 || ld_rt % 8 != 0 || T > (1ll << 30) || C > (1ll << 24))
    return LORA_ERR_UNSUPPORTED_SHAPE;
  if ((reinterpret_cast<uintptr_t>(S) | reinterpret_cast<uintptr_t>(Rt) | reinterpret_cast<uintptr_t>(out)) & 15u)
    return LORA_ERR_MISALIGNED;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNoAllocMaxDevices) return LORA_ERR_NO_DEVICE;
  NoAllocDevice nd;
  {
    // one-time set-up per device (the device is current): resolve the device address of the static array.
    // In host code `g_noalloc_scratch` is only a handle; handing it to a kernel would be a wrong pointer.
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    NoAllocDevice& slot = g_noalloc_dev[dev];
    if (!slot.ready) {
      int major = 0, sms = 0;
      if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess || major != 10)
        return LORA_ERR_NO_DEVICE;
      if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return LORA_ERR_CUDA;
      void* ptr = nullptr;
      if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) {
        cudaGetLastError();
        return LORA_ERR_CUDA;
      }
      if (grad_configure() != cudaSuccess) {
        cudaGetLastError();
        return LORA_ERR_CUDA;
      }
      slot.scratch = static_cast<unsigned char*>(ptr);
      slot.num_sms = sms;
      slot.ready = true;
    }
    nd = slot;
  }
  // grid: the same rule the planned path uses (feature chunks x token chunks, at most one CTA per SM)
  GradParams g{};
  g.T = static_cast<int>(T);
  g.C = static_cast<int>(C);
  g.r = static_cast<int>(r);
  g.r_pad = static_cast<int>((r + 15) / 16 * 16);
  int fc = g.r_pad <= 32 ? 512 : 768;
  const int c128 = static_cast<int>((C + 127) / 128 * 128);
  if (fc > c128) fc = c128;
  g.feat_chunk = fc;
  g.n_feat_chunks = static_cast<int>((C + fc - 1) / fc);
  g.n_slabs = static_cast<int>((T + kGradSlab - 1) / kGradSlab);
  int n_tok = nd.num_sms / g.n_feat_chunks;
  if (n_tok < 1) n_tok = 1;
  if (n_tok > g.n_slabs) n_tok = g.n_slabs;
  g.n_token_chunks = n_tok;
  const size_t fixed = 4 * static_cast<size_t>(g.r_pad) * 128 + 4096;
  int stages = static_cast<int>((232448 - fixed) / kGradStageBytes);
  g.stages = stages > kGradMaxStages ? kGradMaxStages : stages;
  g.c_pad = static_cast<int>((C + 31) / 32 * 32);
  // The partial sums of all token chunks must fit the static array.  One layer (r_pad x c_pad floats) that does not fit
  // is beyond what this entry point serves; otherwise the grid takes as many token chunks as fit, and with a single
  // chunk the kernel needs no partial sums at all (it writes `out` itself), so a fitting shape is never refused, only
  // given fewer CTAs.
  const size_t layer_bytes = static_cast<size_t>(g.r_pad) * g.c_pad * sizeof(float);
  if (kNoAllocHeaderBytes + layer_bytes > kNoAllocScratchBytes) return LORA_ERR_WORKSPACE;
  const int fit = static_cast<int>((kNoAllocScratchBytes - kNoAllocHeaderBytes) / layer_bytes);
  if (n_tok > fit) n_tok = fit >= 2 ? fit : 1;
  g.n_token_chunks = n_tok;
  g.with_p = 0;
  g.side_mn = 0;
  g.do_out = 1;
  g.out_is_da = 0;
  g.scale = 1.0f;
  g.out = static_cast<float*>(out);
  g.out_part = reinterpret_cast<float*>(nd.scratch + kNoAllocHeaderBytes);
  g.p_part = nullptr;
  g.pt_out = nullptr;
  g.ld_t = static_cast<int>(ld_rt);
  g.status = reinterpret_cast<unsigned*>(nd.scratch);
  g.wait_limit = kWaitLimitCycles;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the array keeps the previous call's contents: the status words must start at zero (the partial sums are
  // fully rewritten before they are read)
  if (cudaMemsetAsync(nd.scratch, 0, kNoAllocHeaderBytes, st) != cudaSuccess) return LORA_ERR_CUDA;
  CUtensorMap tmS, tmR;
  if (!noalloc_tmap(&tmS, S, static_cast<uint64_t>(C), static_cast<uint64_t>(T), static_cast<uint64_t>(C), 64, kGradSlab) ||
      !noalloc_tmap(&tmR, Rt, static_cast<uint64_t>(T), static_cast<uint64_t>(r), static_cast<uint64_t>(ld_rt), 64, g.r_pad))
    return LORA_ERR_CUDA;
  if (launch_grad(tmS, tmR, tmR, g, st) != cudaSuccess) return LORA_ERR_CUDA;
  return LORA_OK;
}

extern "C" int lora_grad_contract_noalloc_status(void* stream, int* code) {
  using namespace lora;
  if (code == nullptr) return LORA_ERR_INVALID_ARG;
  *code = LORA_OK;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNoAllocMaxDevices) return LORA_ERR_NO_DEVICE;
  unsigned char* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (g_noalloc_dev[dev].ready) scratch = g_noalloc_dev[dev].scratch;
  }
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return LORA_ERR_CUDA;
  if (scratch == nullptr) return LORA_OK;       // no call was made on this device yet
  unsigned word = 0;                             // a copy into pageable host memory: no allocation on the device
  if (cudaMemcpy(&word, scratch, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return LORA_ERR_CUDA;
  if (word != 0) *code = LORA_ERR_DEVICE_TIMEOUT;
  return LORA_OK;
}

extern "C" int64_t lora_grad_contract_noalloc_max_scratch(void) {
  return static_cast<int64_t>(lora::kNoAllocScratchBytes);
}
