// Dense projection GEMM with the rank-r LoRA adapter fused in (Section 3.2.2, LoRA):
//
//   forward   Y  = X  W^T + s (X  A^T) B^T      act = X,  contraction over d_in
//   backward  dX = dY W   + s (dY B  ) A        act = dY, contraction over d_out
//
// One persistent, warp-specialised kernel per direction:
//   warp 0      TMA producer: 128 x 64 activation tile, block_n x 64 weight tile and the r_pad x 64
//               slice of the adapter's first factor per stage, into a 128-byte-swizzled ring
//   warp 1      issues tcgen05.mma (bf16 -> fp32 in TMEM).  The adapter slice sits directly behind the
//               weight tile in shared memory, so ONE MMA of width block_n + r_pad produces the dense
//               accumulator and act * first-factor (P = X A^T, or Q = dY B) side by side
//   warps 2..5  epilogue: read P/Q from TMEM, scale, round to bf16, write it back to shared memory as
//               an MMA operand; warp 1 then adds (sP) * B^T (or (sQ) * A) with r_pad/16 more MMAs;
//               finally the accumulator is rounded to bf16 and stored with TMA
// Two accumulators live in TMEM (2 x 256 columns), so the epilogue of tile i overlaps the main loop of
// tile i+1; the rank-r MMA of tile i is issued `tail_delay` k-blocks into tile i+1 so that the tensor
// pipe never waits for the bf16 conversion.
//
// Forward operands are all K-major (contraction index contiguous).  In the backward pass W[d_out,d_in],
// B[d_out,r] and A[r,d_in] have the output index contiguous, so they are fed as MN-major operands
// straight from their natural layout: no transposed copy of the frozen weight is kept.
#include "kernels.h"
#include "sm100_ptx.cuh"

namespace lora {

namespace {

struct TileCoord {
  int m_idx, n_idx;
};

__device__ __forceinline__ TileCoord tile_coord(int id, const GemmParams& p) {
  const int per_band = p.group_m * p.tiles_n;
  const int band = id / per_band;
  const int rem = id - band * per_band;
  const int rows = min(p.group_m, p.tiles_m - band * p.group_m);
  TileCoord c;
  c.m_idx = band * p.group_m + rem % rows;
  c.n_idx = rem / rows;
  return c;
}

template <bool kBwd>
__global__ void __launch_bounds__(kGemmThreads, 1)
lora_gemm_kernel(const __grid_constant__ CUtensorMap tm_act,   // X / dY   [M, K]   box 64(k) x 128
                 const __grid_constant__ CUtensorMap tm_w,     // W: fwd box 64(k) x block_n ; bwd box 64(n) x 64(k)
                 const __grid_constant__ CUtensorMap tm_side,  // fwd A box 64(k) x r_pad ; bwd B box 64(r) x 64(k)
                 const __grid_constant__ CUtensorMap tm_tail,  // fwd B box 64(r) x block_n ; bwd A box 64(n) x r_pad
                 const __grid_constant__ CUtensorMap tm_out,   // Y / dX   [M, N]   box 64 x 128
                 const GemmParams p) {
  pdl_launch_dependents();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t ring = smem_u32(smem);
  const uint32_t staging = ring + p.stages * kStageBytes;     // two 16 KiB buffers; [0] doubles as the rank-r operand
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.stages * kStageBytes + 2 * kStagingBytes);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
  auto side_full = [&](int b) { return bar0 + 8u * (2 * kMaxStages + b); };
  auto ps_ready = [&](int b) { return bar0 + 8u * (2 * kMaxStages + 2 + b); };
  auto acc_full = [&](int b) { return bar0 + 8u * (2 * kMaxStages + 4 + b); };
  auto acc_empty = [&](int b) { return bar0 + 8u * (2 * kMaxStages + 6 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kGemmBarriers);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(side_full(b), 1);
      mbar_init(ps_ready(b), 128);
      mbar_init(acc_full(b), 1);
      mbar_init(acc_empty(b), 128);
    }
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tm_act);
    tma_prefetch_desc(&tm_w);
    tma_prefetch_desc(&tm_side);
    tma_prefetch_desc(&tm_tail);
    tma_prefetch_desc(&tm_out);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();                   // global memory of earlier kernels is visible from here on
  const uint32_t tmem_base = *tmem_slot;

  const int G = gridDim.x;
  const int n_my = (p.num_tiles > static_cast<int>(blockIdx.x)) ? (p.num_tiles - 1 - blockIdx.x) / G + 1 : 0;
  const int KB = p.kblocks;
  const int D = min(KB, p.tail_delay);
  const int S = p.stages;
  const int n_groups = p.block_n >> 6;   // 64-column groups of the weight tile (backward layout)

  if (warp == 0) {
    // ================================ TMA producer ================================
    if (lane == 0) {
      int it = 0;
      bool ok = true;
      auto acquire = [&]() -> int {
        const int slot = it % S;
        ok = mbar_wait(empty_bar(slot), ((it / S) & 1) ^ 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_EMPTY);
        ++it;
        return slot;
      };
      auto load_main = [&](int i, int kb) {
        const TileCoord tc = tile_coord(blockIdx.x + i * G, p);
        const int m0 = tc.m_idx * kBlockM, n0 = tc.n_idx * p.block_n, k0 = kb * kBlockK;
        const int slot = acquire();
        if (!ok) return;
        const uint32_t a_dst = ring + slot * kStageBytes, b_dst = a_dst + kStageABytes, fb = full_bar(slot);
        if (!kBwd) {
          mbar_arrive_expect_tx(fb, kStageABytes + (p.block_n + p.r_pad) * 128);
          tma_load_2d(a_dst, &tm_act, fb, k0, m0);
          tma_load_2d(b_dst, &tm_w, fb, k0, n0);
          tma_load_2d(b_dst + p.block_n * 128, &tm_side, fb, k0, 0);
        } else {
          mbar_arrive_expect_tx(fb, kStageABytes + (n_groups + 1) * 8192);
          tma_load_2d(a_dst, &tm_act, fb, k0, m0);
          for (int g = 0; g < n_groups; ++g) tma_load_2d(b_dst + g * 8192, &tm_w, fb, n0 + 64 * g, k0);
          tma_load_2d(b_dst + n_groups * 8192, &tm_side, fb, 0, k0);
        }
      };
      auto load_tail = [&](int i) {
        const TileCoord tc = tile_coord(blockIdx.x + i * G, p);
        const int n0 = tc.n_idx * p.block_n;
        const int slot = acquire();
        if (!ok) return;
        const uint32_t b_dst = ring + slot * kStageBytes + kStageABytes, fb = full_bar(slot);
        if (!kBwd) {
          mbar_arrive_expect_tx(fb, p.block_n * 128);
          tma_load_2d(b_dst, &tm_tail, fb, 0, n0);
        } else {
          mbar_arrive_expect_tx(fb, n_groups * p.r_pad * 128);
          for (int g = 0; g < n_groups; ++g) tma_load_2d(b_dst + g * 8192, &tm_tail, fb, n0 + 64 * g, 0);
        }
      };
      for (int i = 0; i < n_my && ok; ++i) {
        for (int kb = 0; kb < KB && ok; ++kb) {
          if (i > 0 && kb == D) load_tail(i - 1);
          if (ok) load_main(i, kb);
        }
        if (ok && i > 0 && D == KB) load_tail(i - 1);
      }
      if (ok && n_my > 0) load_tail(n_my - 1);
    }
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    if (lane == 0) {
      const uint32_t idesc_main = mma_idesc_bf16(kBlockM, p.block_n + p.r_pad, false, kBwd);
      const uint32_t idesc_tail = mma_idesc_bf16(kBlockM, p.block_n, false, kBwd);
      int it = 0;
      bool ok = true;
      auto mma_main = [&](int i, int kb) {
        const int buf = i & 1, use = i >> 1;
        if (kb == 0) {
          ok = mbar_wait(acc_empty(buf), (use & 1) ^ 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_ACC_EMPTY);
          if (!ok) return;
        }
        const int slot = it % S;
        ok = mbar_wait(full_bar(slot), (it / S) & 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_FULL);
        ++it;
        if (!ok) return;
        tc_fence_after();
        const uint32_t a_addr = ring + slot * kStageBytes, b_addr = a_addr + kStageABytes;
#pragma unroll
        for (int ks = 0; ks < kBlockK / 16; ++ks) {
          const uint64_t ad = smem_desc_sw128(a_addr + ks * 32, 16, 1024);
          const uint64_t bd = kBwd ? smem_desc_sw128(b_addr + ks * 2048, 8192, 1024)
                                   : smem_desc_sw128(b_addr + ks * 32, 16, 1024);
          mma_bf16_ss(tmem_base + buf * 256, ad, bd, idesc_main, (kb | ks) != 0 ? 1u : 0u);
        }
        mma_commit(empty_bar(slot));
        if (kb == KB - 1) mma_commit(side_full(buf));
      };
      auto mma_tail = [&](int i) {
        const int buf = i & 1, use = i >> 1;
        ok = mbar_wait(ps_ready(buf), use & 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_PS);
        if (!ok) return;
        const int slot = it % S;
        ok = mbar_wait(full_bar(slot), (it / S) & 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_FULL);
        ++it;
        if (!ok) return;
        tc_fence_after();
        const uint32_t b_addr = ring + slot * kStageBytes + kStageABytes;
        for (int ks = 0; ks < p.r_pad / 16; ++ks) {
          const uint64_t ad = smem_desc_sw128(staging + ks * 32, 16, 1024);
          const uint64_t bd = kBwd ? smem_desc_sw128(b_addr + ks * 2048, 8192, 1024)
                                   : smem_desc_sw128(b_addr + ks * 32, 16, 1024);
          mma_bf16_ss(tmem_base + buf * 256, ad, bd, idesc_tail, 1u);
        }
        mma_commit(empty_bar(slot));
        mma_commit(acc_full(buf));
      };
      for (int i = 0; i < n_my && ok; ++i) {
        for (int kb = 0; kb < KB && ok; ++kb) {
          if (i > 0 && kb == D) mma_tail(i - 1);
          if (ok) mma_main(i, kb);
        }
        if (ok && i > 0 && D == KB) mma_tail(i - 1);
      }
      if (ok && n_my > 0) mma_tail(n_my - 1);
    }
  } else {
    // ================================ epilogue (128 threads) ================================
    const int e = threadIdx.x - 64;
    const int quarter = warp & 3;                 // TMEM lane quarter this warp may read
    const int row = quarter * 32 + lane;          // tile row == TMEM lane
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    const int n_chunks = p.block_n >> 6;
    for (int i = 0; i < n_my; ++i) {
      const TileCoord tc = tile_coord(blockIdx.x + i * G, p);
      const int m0 = tc.m_idx * kBlockM, n0 = tc.n_idx * p.block_n;
      const int buf = i & 1, use = i >> 1;
      if (e == 0) tma_store_wait_read<0>();       // staging[0] is about to hold the rank-r operand
      bool ok = mbar_wait(side_full(buf), use & 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_SIDE);
      if (named_bar_or(1, 128, !ok)) break;
      tc_fence_after();
      // ---- P (or Q) : TMEM -> scale -> bf16 -> shared memory (K-major, 128-byte swizzle) ----
      for (int c16 = 0; c16 < p.r_pad / 16; ++c16) {
        uint32_t v[16];
        tmem_ld16(lane_addr + buf * 256 + p.block_n + c16 * 16, v);
        tmem_ld_wait();
        uint32_t w[8];
#pragma unroll
        for (int q = 0; q < 8; ++q)
          w[q] = pack_bf16x2(__uint_as_float(v[2 * q]) * p.scale, __uint_as_float(v[2 * q + 1]) * p.scale);
        uint8_t* dst = smem + p.stages * kStageBytes;
        *reinterpret_cast<uint4*>(dst + sw128_offset(row, 2 * c16)) = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4*>(dst + sw128_offset(row, 2 * c16 + 1)) = make_uint4(w[4], w[5], w[6], w[7]);
        if (kBwd && p.rt_out != nullptr && tc.n_idx == 0 && m0 + row < p.M) {
          unsigned short* rt = reinterpret_cast<unsigned short*>(p.rt_out);
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            rt[static_cast<size_t>(c16 * 16 + 2 * q) * p.ld_rt + m0 + row] = static_cast<unsigned short>(w[q] & 0xFFFFu);
            rt[static_cast<size_t>(c16 * 16 + 2 * q + 1) * p.ld_rt + m0 + row] = static_cast<unsigned short>(w[q] >> 16);
          }
        }
      }
      fence_proxy_async_smem();
      tc_fence_before();
      mbar_arrive(ps_ready(buf));
      // ---- accumulator: TMEM -> bf16 -> swizzled staging -> TMA store, 64 columns at a time ----
      ok = mbar_wait(acc_full(buf), use & 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_ACC);
      if (named_bar_or(1, 128, !ok)) break;
      tc_fence_after();
      for (int c = 0; c < n_chunks; ++c) {
        uint32_t v0[32], v1[32];
        tmem_ld32(lane_addr + buf * 256 + c * 64, v0);
        tmem_ld32(lane_addr + buf * 256 + c * 64 + 32, v1);
        tmem_ld_wait();
        if (c == n_chunks - 1) {
          tc_fence_before();
          mbar_arrive(acc_empty(buf));
        }
        if (n0 + c * 64 >= p.N) continue;           // whole chunk right of the matrix (uniform)
        if (e == 0) tma_store_wait_read<1>();       // the store issued two chunks ago has left its buffer
        named_bar_sync(2, 128);
        uint8_t* dst = smem + p.stages * kStageBytes + (c & 1) * kStagingBytes;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint4 w;
          w.x = pack_bf16x2(__uint_as_float(v0[8 * q + 0]), __uint_as_float(v0[8 * q + 1]));
          w.y = pack_bf16x2(__uint_as_float(v0[8 * q + 2]), __uint_as_float(v0[8 * q + 3]));
          w.z = pack_bf16x2(__uint_as_float(v0[8 * q + 4]), __uint_as_float(v0[8 * q + 5]));
          w.w = pack_bf16x2(__uint_as_float(v0[8 * q + 6]), __uint_as_float(v0[8 * q + 7]));
          *reinterpret_cast<uint4*>(dst + sw128_offset(row, q)) = w;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint4 w;
          w.x = pack_bf16x2(__uint_as_float(v1[8 * q + 0]), __uint_as_float(v1[8 * q + 1]));
          w.y = pack_bf16x2(__uint_as_float(v1[8 * q + 2]), __uint_as_float(v1[8 * q + 3]));
          w.z = pack_bf16x2(__uint_as_float(v1[8 * q + 4]), __uint_as_float(v1[8 * q + 5]));
          w.w = pack_bf16x2(__uint_as_float(v1[8 * q + 6]), __uint_as_float(v1[8 * q + 7]));
          *reinterpret_cast<uint4*>(dst + sw128_offset(row, 4 + q)) = w;
        }
        fence_proxy_async_smem();
        named_bar_sync(2, 128);
        if (e == 0) {
          tma_store_2d(&tm_out, staging + (c & 1) * kStagingBytes, n0 + c * 64, m0);
          tma_store_commit();
        }
      }
    }
    if (e == 0) tma_store_wait_all<0>();
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
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

size_t gemm_smem_bytes(int stages) {
  return static_cast<size_t>(stages) * kStageBytes + 2 * kStagingBytes + kGemmBarriers * 8 + 16 + 1024;
}

cudaError_t gemm_configure() {
  cudaError_t e = cudaFuncSetAttribute(lora_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(gemm_smem_bytes(4)));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(lora_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(gemm_smem_bytes(4)));
}

cudaError_t launch_gemm_fwd(const CUtensorMap& tmX, const CUtensorMap& tmW, const CUtensorMap& tmA,
                            const CUtensorMap& tmB, const CUtensorMap& tmY, const GemmParams& p, int ctas,
                            cudaStream_t stream) {
  return launch_pdl(lora_gemm_kernel<false>, dim3(ctas), dim3(kGemmThreads), gemm_smem_bytes(p.stages), stream, tmX, tmW, tmA,
                    tmB, tmY, p);
}

cudaError_t launch_gemm_dx(const CUtensorMap& tmdY, const CUtensorMap& tmW, const CUtensorMap& tmB,
                           const CUtensorMap& tmA, const CUtensorMap& tmdX, const GemmParams& p, int ctas,
                           cudaStream_t stream) {
  return launch_pdl(lora_gemm_kernel<true>, dim3(ctas), dim3(kGemmThreads), gemm_smem_bytes(p.stages), stream, tmdY, tmW, tmB,
                    tmA, tmdX, p);
}

}  // namespace lora
