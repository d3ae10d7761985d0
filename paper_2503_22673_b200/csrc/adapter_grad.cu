// Adapter gradients of the LoRA layer (Section 3.2.2, LoRA): tall-skinny contractions over the tokens.
//
//   dA = s (dY B)^T X      streams X  [T, d_in]  once, second factor Qt = s (dY B)^T  [r_pad, T] (bf16)
//   dB = s dY^T (X A^T)    streams dY [T, d_out] once, second factor Pt = s (X A^T)^T [r_pad, T] (bf16)
//
// Both are out[c, j] = sum_t S[t, c] * Rt[j, t]: the streamed matrix S is the MN-major A operand of a
// tcgen05 MMA (M = 128 features, N = r_pad, K = tokens) read from the very 128-byte-swizzled tiles TMA
// delivers, so the token reduction runs on the tensor cores while the kernel stays bound by the HBM
// stream.  The same tiles, read as the K-major operand with M = 128 tokens, give the SIDE product
// S side^T of the slab: X A^T inside the dA launch (the backward pass is not given the forward's X A^T), or dY B.
// The side operand has two forms: A [r, C] (K-major rows) or B [C, r] (MN-major, its natural layout); with
// do_out = 0 the kernel computes only the side product (the X A^T and dY B pre-passes of the K-extended GEMMs).
//
// Grid: (feature chunks, token chunks), one CTA per SM, ONE launch, no CTA outside a cluster ever waits for another.
//  * Gradient: a CTA keeps feat_chunk x r_pad fp32 sums in TMEM over all slabs of its token chunk.  The token chunks
//    of one feature chunk form a thread-block cluster (up to 16 CTAs along y).  At the end every CTA copies its sums
//    to its own shared memory, the cluster synchronises, and CTA k of the cluster adds slice k of all copies over
//    distributed shared memory IN RANK ORDER and writes that slice of dA / dB: bitwise reproducible, no partial sums
//    in global memory, no second launch.
//  * Side product: a CTA holds only its feature chunk's share of a slab's X A^T.  With one feature chunk it writes
//    the bf16 result itself; otherwise it writes an fp32 partial, bumps the slab's arrival counter, and the CTA that
//    arrives last adds the partials IN CHUNK ORDER, scales, rounds and writes the slab (and resets the counter).
//
// Warps: 0..3 TMA producers of the streamed tiles (ring items round-robin: one warp's copies sustain only ~37 B/clk),
// 4 MMA issuer + TMEM, 5 loader of the second factor, 6..9 and 10..13 two epilogue groups (slabs alternate between them,
// so that the fence + atomic round trip of one slab's side product overlaps the next slab's drain).
#include "kernels.h"
#include "sm100_ptx.cuh"

#include <mutex>

#include "../../include/lora_linear.h"

namespace lora {

namespace {

constexpr int kGradBarriers = 2 * kGradMaxStages + 2 * kGradMaxRtBufs + 2 * kGradPBufs + 1;
constexpr int kGradTailBytes = kGradBarriers * 8 + 32;      // barriers, TMEM slot, abort flag, two broadcast words
constexpr int kGradMmaWarp = kGradProducerWarps;
constexpr int kGradLoaderWarp = kGradProducerWarps + 1;
constexpr int kGradEpiWarp0 = kGradProducerWarps + 2;
constexpr int kGradEpiThreads = 128 * kGradEpiGroups;

__device__ __forceinline__ float4 ld_cluster_f4(uint32_t cluster_addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(cluster_addr) : "memory");
  return v;
}

// One launch runs up to kGradMaxJobs JOBS side by side (e.g. dA over X next to dB over dY, or X A^T next to dY B; the
// grouped projections add one job per group): CTAs with blockIdx.x in [x_end[j-1], x_end[j]) belong to job j.  A job's
// CTAs are numbered (feature chunk, token chunk): with a gradient the token chunk is blockIdx.y (= rank in the cluster),
// otherwise both indices are folded into x.  maps.m[3 j + 0 .. 2] = job j's streamed matrix [T, C] box 64(c) x 128(t),
// second factor [r_pad, T] box 64(t) x r_pad, side operand (with_p): A [r, C] box 64(c) x r_pad, or B [C, r] box
// 64(r, zero-filled) x 64(c) when side_mn.
__global__ void __launch_bounds__(kGradThreads, 1)
lora_grad_kernel(const __grid_constant__ GradMaps maps, const __grid_constant__ GradLaunch L) {
  pdl_launch_dependents();
  int job = 0;
  while (job + 1 < L.n_jobs && static_cast<int>(blockIdx.x) >= L.x_end[job]) ++job;
  const GradParams p = L.job[job];
  const CUtensorMap& tm_s = maps.m[3 * job];
  const CUtensorMap& tm_r = maps.m[3 * job + 1];
  const CUtensorMap& tm_a = maps.m[3 * job + 2];
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int NB = p.feat_chunk >> 7;                 // 128-feature accumulator blocks of a full chunk
  const int rt_box = p.r_pad * 128;                 // bytes of one 64-wide box with r_pad rows
  const int side_box = p.side_mn ? 8192 : rt_box;   // bytes of the side operand for 64 features
  // A gradient CTA with ONE block and no side product needs a new slab of the second factor with every tile: the slab then
  // travels in the tile's own stage (same barrier, same producer), and the loader warp and its ring are idle.
  const bool rt_in_stage = p.rt_in_stage != 0;
  const int stage_bytes = kGradStageBytes + (p.with_p ? 2 * side_box : 0) + (rt_in_stage ? 2 * rt_box : 0);
  const int ring_bytes = p.stages * stage_bytes;
  const uint32_t ring = smem_u32(smem);
  const uint32_t rt_base = ring + ring_bytes;                           // rt_bufs buffers x 2 boxes of the second factor
  const int RB = p.rt_bufs;
  uint8_t* tail = smem + ring_bytes + 2 * RB * rt_box;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tail);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kGradMaxStages + s); };
  auto rt_full = [&](int b) { return bar0 + 8u * (2 * kGradMaxStages + b); };
  auto rt_empty = [&](int b) { return bar0 + 8u * (2 * kGradMaxStages + kGradMaxRtBufs + b); };
  auto p_full = [&](int b) { return bar0 + 8u * (2 * kGradMaxStages + 2 * kGradMaxRtBufs + b); };
  auto p_empty = [&](int b) { return bar0 + 8u * (2 * kGradMaxStages + 2 * kGradMaxRtBufs + kGradPBufs + b); };
  const uint32_t out_full = bar0 + 8u * (2 * kGradMaxStages + 2 * kGradMaxRtBufs + 2 * kGradPBufs);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kGradBarriers);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* epi_word = reinterpret_cast<volatile int*>(tmem_slot + 2);      // one broadcast word per epilogue group

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int local_x = static_cast<int>(blockIdx.x) - (job > 0 ? L.x_end[job - 1] : 0);
  const int fc = p.do_out ? local_x : local_x % p.n_feat_chunks;
  const int tc = p.do_out ? static_cast<int>(blockIdx.y) : local_x / p.n_feat_chunks;
  const int c0 = fc * p.feat_chunk;
  const int nb_count = min(NB, (p.C - c0 + 127) >> 7);          // blocks of THIS chunk (the last chunk may be short)
  const int s_begin = static_cast<int>(static_cast<long long>(tc) * p.n_slabs / p.n_token_chunks);
  const int s_end = static_cast<int>(static_cast<long long>(tc + 1) * p.n_slabs / p.n_token_chunks);
  const int S = p.stages;
  bool alive = true;            // false once a bounded wait of this thread's role gave up

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < RB; ++b) {
      mbar_init(rt_full(b), 1);
      mbar_init(rt_empty(b), 1);
    }
    for (int b = 0; b < kGradPBufs; ++b) {
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
  if (warp == kGradMmaWarp) {
    tmem_alloc(smem_u32(tmem_slot), p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();                   // global memory of earlier kernels is visible from here on
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_p = tmem_base + (p.do_out ? NB * p.r_pad : 0);     // kGradPBufs r_pad-column buffers for the side product

  if (warp < kGradProducerWarps) {
    // ================================ TMA producers: streamed tiles, ring items round-robin ================================
    // At most S warps take part.  A producer that waits for the k-th release of a slot relies on the (k-1)-th having
    // happened (the wait only sees the parity of the phase): its previous item, PW items back, guarantees that only
    // when PW <= S.
    const int PW = min(kGradProducerWarps, S);
    int slot = 0, phase = 0, turn = 0;
    bool ok = warp < PW;
    for (int s = s_begin; s < s_end && ok; ++s) {
      const int t0 = s * kGradSlab;
      for (int nb = 0; nb < nb_count && ok; ++nb) {
        if (turn == warp) {
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
            } else if (rt_in_stage) {
              tma_load_2d(dst + 32768, &tm_r, fb, t0, 0);
              tma_load_2d(dst + 32768 + rt_box, &tm_r, fb, t0 + 64, 0);
            }
          }
          __syncwarp();
        }
        if (++slot == S) { slot = 0; phase ^= 1; }
        if (++turn == PW) turn = 0;
      }
    }
  } else if (warp == kGradLoaderWarp) {
    // ================================ loader of the second factor (one 128-token slab at a time) ================================
    bool ok = true;
    int rb = 0, rphase = 0;
    for (int s = s_begin; s < s_end && ok && p.do_out && !rt_in_stage && !p.debug_no_second_factor; ++s) {
      ok = warp_wait(rt_empty(rb), rphase ^ 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_EMPTY, false, 20);
      if (ok && elect_one()) {
        const int t0 = s * kGradSlab;
        mbar_arrive_expect_tx(rt_full(rb), 2 * rt_box);
        tma_load_2d(rt_base + (2 * rb) * rt_box, &tm_r, rt_full(rb), t0, 0);
        tma_load_2d(rt_base + (2 * rb + 1) * rt_box, &tm_r, rt_full(rb), t0 + 64, 0);
      }
      __syncwarp();
      if (++rb == RB) { rb = 0; rphase ^= 1; }
    }
  } else if (warp == kGradMmaWarp) {
    // ================================ MMA issuer ================================
    const uint32_t idesc_out = mma_idesc_bf16(128, p.r_pad, true, false);   // A operand = S tile, MN-major
    const uint32_t idesc_p = mma_idesc_bf16(128, p.r_pad, false, p.side_mn != 0);   // A operand = S tile, K-major
    const uint64_t a_mn0 = smem_desc_sw128(ring, 16384, 1024);              // S tile as [features x tokens]
    const uint64_t a_k0 = smem_desc_sw128(ring, 16, 1024);                  // S tile as [tokens x features]
    const uint64_t w_k0 = smem_desc_sw128(ring + 32768, 16, 1024);          // side operand of the stage
    const uint32_t sbox = static_cast<uint32_t>(side_box) >> 4;
    const uint32_t sstep = p.side_mn ? 128u : 2u;                           // descriptor step per 16 features
    const uint64_t r_k0 = smem_desc_sw128(rt_in_stage ? ring + 32768 : rt_base, 16, 1024);   // second factor
    bool ok = true;
    int slot = 0, phase = 0, rb = 0, rphase = 0, pb = 0, pphase = 0;
    for (int s = s_begin; s < s_end && ok; ++s) {
      if (p.do_out && !rt_in_stage)
        ok = warp_wait(rt_full(rb), rphase, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_FULL, false, 0);
      if (ok && p.with_p)
        ok = warp_wait(p_empty(pb), pphase ^ 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_ACC_EMPTY, false, 0);
      for (int nb = 0; nb < nb_count && ok; ++nb) {
        ok = warp_wait(full_bar(slot), phase, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_FULL, false, 0);
        if (!ok) break;
        tc_fence_after();
        if (elect_one()) {
          const uint32_t so = static_cast<uint32_t>(slot * stage_bytes) >> 4;
          const uint32_t ro = rt_in_stage ? so : static_cast<uint32_t>(2 * rb * rt_box) >> 4;
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
              mma_bf16_ss(tmem_p + pb * p.r_pad, a_k0 + so + (kk >> 2) * 1024 + (kk & 3) * 2,
                          w_k0 + so + (kk >> 2) * sbox + (kk & 3) * sstep, idesc_p, (nb != 0 || kk != 0) ? 1u : 0u);
          }
          mma_commit(empty_bar(slot));
          if (nb == nb_count - 1) {
            if (p.do_out && !rt_in_stage) mma_commit(rt_empty(rb));
            if (p.with_p) mma_commit(p_full(pb));
          }
        }
        __syncwarp();
        if (++slot == S) { slot = 0; phase ^= 1; }
      }
      if (++rb == RB) { rb = 0; rphase ^= 1; }
      if (++pb == kGradPBufs) { pb = 0; pphase ^= 1; }
    }
    if (ok && p.do_out && elect_one()) mma_commit(out_full);
    __syncwarp();
  } else {
    // ================================ epilogue (two groups of four warps) ================================
    const int grp = (warp - kGradEpiWarp0) >> 2;
    const int quarter = warp & 3;                  // the TMEM lane quarter a warp may read is fixed by its index
    const int row = quarter * 32 + lane;
    const int gtid = (warp - kGradEpiWarp0 - 4 * grp) * 32 + lane;
    const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
    const int bar_id = 1 + grp;
    if (p.with_p) {
      // ---- the side product of each slab: this CTA's share over its features ----
      int ls = 0;
      for (int s = s_begin; s < s_end; ++s, ++ls) {
        if ((ls & (kGradEpiGroups - 1)) != grp) continue;
        const int pb = ls & (kGradPBufs - 1), pphase = (ls / kGradPBufs) & 1;
        const int t = s * kGradSlab + row;
        bool ok = warp_wait(p_full(pb), pphase, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_SIDE, false, 32);
        if (named_bar_or(bar_id, 128, !ok)) { alive = false; break; }
        tc_fence_after();
        for (int c16 = 0; c16 < p.r_pad / 16; ++c16) {
          uint32_t v[16];
          tmem_ld16(tmem_p + lane_addr + pb * p.r_pad + c16 * 16, v);
          tmem_ld_wait();
          if (t < p.T && p.n_feat_chunks > 1) {
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
        if (p.n_feat_chunks > 1) {
          // The group's partials must be visible device-wide before its arrival is counted: the barrier orders every
          // thread's stores before thread 0's fence, and a fence is cumulative over what its thread has synchronised with.
          named_bar_sync(bar_id, 128);
          if (gtid == 0) {
            __threadfence();
            epi_word[grp] = atomicAdd(p.side_count + s, 1);
          }
          named_bar_sync(bar_id, 128);
          if (epi_word[grp] == p.n_feat_chunks - 1) {
            // last feature chunk to arrive for this slab: add all partials in chunk order
            __threadfence();
            if (t < p.T) {
              unsigned short* pt = reinterpret_cast<unsigned short*>(p.pt_out);
              for (int j0 = 0; j0 < p.r_pad; j0 += 16) {
                float acc[16];
#pragma unroll
                for (int q = 0; q < 16; ++q) acc[q] = 0.f;
                for (int f = 0; f < p.n_feat_chunks; ++f) {
                  const float* src = p.p_part + (static_cast<size_t>(f) * p.r_pad + j0) * p.ld_t + t;
                  float v[16];
#pragma unroll
                  for (int q = 0; q < 16; ++q) v[q] = __ldcg(src + static_cast<size_t>(q) * p.ld_t);
#pragma unroll
                  for (int q = 0; q < 16; ++q) acc[q] += v[q];
                }
#pragma unroll
                for (int q = 0; q < 16; ++q)
                  pt[static_cast<size_t>(j0 + q) * p.ld_t + t] =
                      static_cast<unsigned short>(pack_bf16x2(acc[q] * p.scale, 0.f) & 0xFFFFu);
              }
            }
            if (gtid == 0) p.side_count[s] = 0;          // ready for the next launch
          }
        }
      }
    }
    if (alive && p.do_out) {
      const bool ok = warp_wait(out_full, 0, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_ACC, false, 32);
      if (named_bar_or(bar_id, 128, !ok)) alive = false;
      tc_fence_after();
    }
  }

  // ================================ gradient: sum over the token chunks inside the cluster ================================
  // Every thread of every CTA of the cluster passes the same cluster barriers (all loop bounds are launch constants).
  if (p.do_out) {
    const int CS = p.n_token_chunks;                       // = cluster size along y, so cluster rank = tc
    int bpp = ring_bytes / (p.r_pad * 512);                // blocks whose sums fit into the (now idle) ring at once
    if (bpp < 1) bpp = 1;
    float* stage_f = reinterpret_cast<float*>(smem);
    for (int b0 = 0; b0 < nb_count; b0 += bpp) {
      const int b1 = min(nb_count, b0 + bpp);
      if (warp >= kGradEpiWarp0 && alive && !*abort_flag) {
        // ---- TMEM -> this CTA's shared memory (blocks alternate between the two epilogue groups) ----
        const int grp = (warp - kGradEpiWarp0) >> 2;
        const int row = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
        for (int nb = b0 + grp; nb < b1; nb += kGradEpiGroups) {
          const int nbl = nb - b0;
          for (int c16 = 0; c16 < p.r_pad / 16; ++c16) {
            uint32_t v[16];
            tmem_ld16(tmem_base + lane_addr + nb * p.r_pad + c16 * 16, v);
            tmem_ld_wait();
            if (p.out_is_da) {        // [block][j][feature]
#pragma unroll
              for (int q = 0; q < 16; ++q) stage_f[(nbl * p.r_pad + c16 * 16 + q) * 128 + row] = __uint_as_float(v[q]);
            } else {                  // [block][feature][j]
              float4* dst = reinterpret_cast<float4*>(stage_f + (nbl * 128 + row) * p.r_pad + c16 * 16);
#pragma unroll
              for (int q = 0; q < 4; ++q)
                dst[q] = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]), __uint_as_float(v[4 * q + 2]),
                                     __uint_as_float(v[4 * q + 3]));
            }
          }
        }
      }
      cluster_sync_all();            // every CTA's copy is complete and visible to the cluster
      if (warp >= kGradEpiWarp0 && !*abort_flag) {
        // ---- CTA k adds slice k of all copies, in rank order, and writes that slice of the gradient ----
        const int tot4 = (b1 - b0) * p.r_pad * 32;         // float4 groups of this pass
        const int n4 = (tot4 + CS - 1) / CS;               // ... per CTA of the cluster (the last slice may be short)
        const int etid = threadIdx.x - kGradEpiWarp0 * 32;
        for (int i = etid; i < n4 && tc * n4 + i < tot4; i += kGradEpiThreads) {
          const int q4 = tc * n4 + i;
          const uint32_t off = static_cast<uint32_t>(q4) * 16u;
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
          for (int rr = 0; rr < CS; ++rr) {
            const float4 v = ld_cluster_f4(map_to_cta(ring + off, static_cast<uint32_t>(rr)));
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
          }
          const int e = q4 * 4;
          if (p.out_is_da) {
            const int rowc = e & 127, jj = (e >> 7) % p.r_pad, nbl = (e >> 7) / p.r_pad;
            const int c = c0 + (b0 + nbl) * 128 + rowc;
            if (jj < p.r && c < p.C) {
              float4* dst = reinterpret_cast<float4*>(p.out + static_cast<size_t>(jj) * p.C + c);
              if (p.accumulate) { const float4 o = *dst; acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w; }
              *dst = acc;
            }
          } else {
            const int jj = e % p.r_pad, rowc = (e / p.r_pad) & 127, nbl = e / (p.r_pad * 128);
            const int c = c0 + (b0 + nbl) * 128 + rowc;
            if (jj < p.r && c < p.C) {
              float4* dst = reinterpret_cast<float4*>(p.out + static_cast<size_t>(c) * p.r + jj);
              if (p.accumulate) { const float4 o = *dst; acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w; }
              *dst = acc;
            }
          }
        }
      }
      cluster_sync_all();            // no CTA overwrites its copy, or leaves, while a peer may still read it
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
  if (warp == kGradMmaWarp) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

}  // namespace

size_t grad_smem_bytes(const GradParams& p) {
  const size_t stage = kGradStageBytes + (p.with_p ? 2 * (p.side_mn ? size_t(8192) : static_cast<size_t>(p.r_pad) * 128) : 0) +
                       (p.rt_in_stage ? 2 * static_cast<size_t>(p.r_pad) * 128 : 0);
  return static_cast<size_t>(p.stages) * stage + 2 * static_cast<size_t>(p.rt_bufs) * p.r_pad * 128 + kGradTailBytes + 1024;
}

void grad_set_ring(GradParams* p) {
  const bool in_stage = p->do_out && !p->with_p && p->feat_chunk == 128 && !p->debug_no_second_factor;
  p->rt_in_stage = in_stage ? 1 : 0;
  p->rt_bufs = !p->do_out ? 1 : (in_stage ? 1 : (p->r_pad <= 32 ? 4 : 3));
  const size_t side_box = p->side_mn ? size_t(8192) : static_cast<size_t>(p->r_pad) * 128;
  const size_t stage = kGradStageBytes + (p->with_p ? 2 * side_box : 0) + (in_stage ? 2 * static_cast<size_t>(p->r_pad) * 128 : 0);
  const size_t fixed = 2 * static_cast<size_t>(p->rt_bufs) * p->r_pad * 128 + kGradTailBytes + 1024;
  int stages = static_cast<int>((232448 - fixed) / stage);
  if (stages > kGradMaxStages) stages = kGradMaxStages;
  p->stages = stages < 2 ? 2 : stages;
}

cudaError_t grad_configure() {
  cudaError_t e = cudaFuncSetAttribute(lora_grad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(lora_grad_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
  return e;
}

int grad_max_resident_ctas(int cluster, size_t smem_bytes) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(1, static_cast<unsigned>(cluster), 1);
  cfg.blockDim = dim3(kGradThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1;
  attr[0].val.clusterDim.y = static_cast<unsigned>(cluster);
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, lora_grad_kernel, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n * cluster;
}

GradGrid grad_pick_grid(long long T, long long C, long long C2, int r_pad, bool with_p, bool side_mn, const int* caps) {
  const long long cs[2] = {C, C2};
  return grad_pick_grid_jobs(T, cs, C2 > 0 ? 2 : 1, r_pad, with_p, side_mn, caps);
}

GradGrid grad_pick_grid_jobs(long long T, const long long* C, int n_jobs, int r_pad, bool with_p, bool side_mn, const int* caps) {
  int nblk_sum = 0, nblk_max = 0;
  for (int j = 0; j < n_jobs; ++j) {
    const int b = static_cast<int>((C[j] + 127) / 128);
    nblk_sum += b;
    if (b > nblk_max) nblk_max = b;
  }
  auto chunks = [&](int nb) {
    int n = 0;
    for (int j = 0; j < n_jobs; ++j) n += (static_cast<int>((C[j] + 127) / 128) + nb - 1) / nb;
    return n;
  };
  const int n_slabs = static_cast<int>((T + kGradSlab - 1) / kGradSlab);
  int nb_max = (512 - (with_p ? kGradPBufs * r_pad : 0)) / r_pad;          // TMEM: NB x r_pad + side buffers <= 512 columns
  if (nb_max < 1) nb_max = 1;
  if (nb_max > nblk_max) nb_max = nblk_max;
  GradGrid best{};
  double best_t = 1e300;
  for (int cs = 1; cs <= kGradMaxCluster; ++cs) {
    if (cs > n_slabs || caps[cs] < cs) continue;
    const int slabs_per = (n_slabs + cs - 1) / cs;
    for (int nb = 1; nb <= nb_max; ++nb) {
      const int n_feat = chunks(nb);
      if (n_feat * cs > caps[cs]) continue;
      // time in tile units (one 128 x 128 tile of the stream): the busiest CTA's tiles, but never less than the stream
      // needs when every SM pulls its share of the HBM bandwidth (about 120 busy SMs saturate it); side-product partial
      // sums add r_pad / (32 nb) of a tile's bytes per tile (written and read back); a cluster reduction ~1.5 tiles
      double t = static_cast<double>(nb) * slabs_per;
      const double sat = static_cast<double>(nblk_sum) * n_slabs / 120.0;
      if (t < sat) t = sat;
      if (with_p && n_feat > 1) t *= 1.0 + r_pad / (32.0 * nb);
      if (cs > 1) t += 1.5;
      if (t < best_t - 1e-9) {
        best_t = t;
        best.feat_chunk = nb * 128;
        best.n_feat = n_feat;
        best.n_tok = cs;
      }
    }
  }
  if (best.feat_chunk == 0) {
    // more feature chunks than CTAs are resident at once even at the widest chunk: widest chunk, no cluster, several waves
    best.feat_chunk = nb_max * 128;
    best.n_feat = chunks(nb_max);
    best.n_tok = 1;
  }
  const size_t side_box = side_mn ? size_t(8192) : static_cast<size_t>(r_pad) * 128;
  const size_t stage = kGradStageBytes + (with_p ? 2 * side_box : 0);
  {
    GradParams t{};
    t.do_out = 1;
    t.with_p = with_p ? 1 : 0;
    t.side_mn = side_mn ? 1 : 0;
    t.r_pad = r_pad;
    t.feat_chunk = best.feat_chunk;
    grad_set_ring(&t);
    best.stages = t.stages;
  }
  best.tmem_cols = grad_tmem_cols(best.feat_chunk, r_pad, true, with_p);
  return best;
}

int grad_tmem_cols(int feat_chunk, int r_pad, bool do_out, bool with_p) {
  const int need = (do_out ? (feat_chunk / 128) * r_pad : 0) + (with_p ? kGradPBufs * r_pad : 0);
  int cols = 32;
  while (cols < need) cols <<= 1;
  return cols;
}

void grad_default_caps(int num_sms, int* caps) {
  // Without a device to ask: SMs come in groups of about 18 (a GPC), a cluster must fit inside one group, and the largest
  // clusters find room in all but one group
  const int groups = num_sms / 18 > 0 ? num_sms / 18 : 1;
  caps[0] = 0;
  for (int cs = 1; cs <= kGradMaxCluster; ++cs) {
    int cap = (cs > 8 && groups > 1 ? groups - 1 : groups) * ((18 / cs) * cs);
    if (cap > num_sms / cs * cs) cap = num_sms / cs * cs;
    caps[cs] = cs == 1 ? num_sms : cap;
  }
}

void grad_device_caps(int num_sms, int* caps) {
  caps[0] = 0;
  caps[1] = num_sms;
  for (int cs = 2; cs <= kGradMaxCluster; ++cs) caps[cs] = grad_max_resident_ctas(cs, 232448);
}

cudaError_t launch_grad_jobs(const GradJobDesc* jobs, int n_jobs, cudaStream_t stream) {
  if (n_jobs < 1 || n_jobs > kGradMaxJobs) return cudaErrorInvalidValue;
  GradMaps maps;
  GradLaunch L{};
  L.n_jobs = n_jobs;
  const int do_out = jobs[0].p.do_out;
  const int cluster = do_out ? jobs[0].p.n_token_chunks : 1;
  size_t smem = 0;
  int x = 0;
  for (int j = 0; j < n_jobs; ++j) {
    GradParams p = jobs[j].p;
    // all jobs of a launch share the cluster shape: all compute a gradient with the same number of token chunks, or none does
    if (p.do_out != do_out || (do_out && p.n_token_chunks != cluster)) return cudaErrorInvalidValue;
    grad_set_ring(&p);                    // ring depth, second-factor ring / in-stage slab: one rule for every caller
    L.job[j] = p;
    maps.m[3 * j] = jobs[j].tmS;
    maps.m[3 * j + 1] = jobs[j].tmR;
    maps.m[3 * j + 2] = jobs[j].tmSide;
    // x extent of a job: feature chunks (gradient: the token chunks are the cluster along y) or feature x token chunks
    x += do_out ? p.n_feat_chunks : p.n_feat_chunks * p.n_token_chunks;
    L.x_end[j] = x;
    if (grad_smem_bytes(p) > smem) smem = grad_smem_bytes(p);
  }
  for (int j = n_jobs; j < kGradMaxJobs; ++j) {
    L.x_end[j] = x;
    maps.m[3 * j] = maps.m[3 * j + 1] = maps.m[3 * j + 2] = jobs[0].tmS;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(x), static_cast<unsigned>(cluster), 1);
  cfg.blockDim = dim3(kGradThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.numAttrs = 1;
  if (cluster > 1) {
    // the token chunks of a feature chunk are one cluster: their gradient sums meet in distributed shared memory
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = static_cast<unsigned>(cluster);
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  cfg.attrs = attr;
  return cudaLaunchKernelEx(&cfg, lora_grad_kernel, maps, L);
}

cudaError_t launch_grad(const CUtensorMap& tmS, const CUtensorMap& tmR, const CUtensorMap& tmA, const GradParams& p,
                        cudaStream_t stream) {
  GradJobDesc j;
  j.tmS = tmS;
  j.tmR = tmR;
  j.tmSide = tmA;
  j.p = p;
  return launch_grad_jobs(&j, 1, stream);
}

// ================================================================================================
// No-allocation variant of the dB-style contraction: scratch lives in a static device array
// ================================================================================================
namespace {

// Scratch held by every GPU that loads this library, until the process exits.  The contraction kernel sums its
// token chunks on chip (thread-block cluster), so the only global scratch it needs is its status block.
constexpr size_t kNoAllocScratchBytes = 4096;
constexpr size_t kNoAllocHeaderBytes = 4096;     // [0,256) status words, rest reserved
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

struct NoAllocDevice {
  bool ready = false;
  unsigned char* scratch = nullptr;   // device address of g_noalloc_scratch on this device
  int caps[kGradMaxCluster + 1] = {};  // CTAs resident at once for clusters of 1 .. 16 CTAs
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
      grad_device_caps(sms, slot.caps);
      slot.ready = true;
    }
    nd = slot;
  }
  // grid: the same rule the planned path uses (feature chunks x one cluster of token chunks)
  GradParams g{};
  g.T = static_cast<int>(T);
  g.C = static_cast<int>(C);
  g.r = static_cast<int>(r);
  g.r_pad = static_cast<int>((r + 15) / 16 * 16);
  const GradGrid gg = grad_pick_grid(T, C, 0, g.r_pad, false, false, nd.caps);
  g.feat_chunk = gg.feat_chunk;
  g.n_feat_chunks = gg.n_feat;
  g.n_token_chunks = gg.n_tok;
  g.n_slabs = static_cast<int>((T + kGradSlab - 1) / kGradSlab);
  g.tmem_cols = gg.tmem_cols;
  g.with_p = 0;
  g.side_mn = 0;
  g.do_out = 1;
  g.out_is_da = 0;
  g.scale = 1.0f;
  g.out = static_cast<float*>(out);
  g.p_part = nullptr;
  g.side_count = nullptr;
  g.pt_out = nullptr;
  g.ld_t = static_cast<int>(ld_rt);
  g.status = reinterpret_cast<unsigned*>(nd.scratch);
  g.wait_limit = kWaitLimitCycles;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the array keeps the previous call's contents: the status words must start at zero
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
