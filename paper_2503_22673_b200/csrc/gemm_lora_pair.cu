// CTA-pair variant of the dense projection GEMM with the rank-r LoRA adapter fused in (Section 3.2.2, LoRA):
//
//   forward   Y  = X  W^T + s (X  A^T) B^T      act = X,  contraction over d_in
//   backward  dX = dY W   + s (dY B  ) A        act = dY, contraction over d_out
//
// Two CTAs on the two SMs of a TPC (cluster of 2) own one 256 x block_n output tile.  Each CTA stages its own
// 128 activation rows and HALF of the weight tile; one tcgen05.mma.cta_group::2 (M = 256) issued by the leader
// CTA reads both shared memories, so every weight byte is fetched from L2 once per 256 rows instead of once per
// 128.  That halves the L2 -> shared-memory traffic per FLOP, which is what bounds the single-CTA kernel.
// No TMA multicast is used anywhere: each CTA issues plain loads for its own half.
//
// Roles per CTA: warps 0..3 TMA producers (both CTAs), warp 4 MMA issuer (leader only) + TMEM allocation,
// warps 5..8 epilogue (both CTAs, 128 rows each).  One warp's TMA copies sustain only ~30 B/clk (measured),
// far below what the tensor pipe consumes, while copies from different warps proceed in parallel: so the
// activation tile and the weight tile are issued by different warps, and even / odd ring items by different
// warp pairs.  Barriers:
//   full[s]      leader's, 2 arrivals (its activation and its weight producer), each arming the byte count of
//                that operand for BOTH CTAs; both CTAs' loads credit it
//   empty[s]     per CTA; tcgen05.commit multicast to both CTAs when the MMAs that read the stage are done
//   side_full[b] per CTA; commit multicast: P (or Q) columns of accumulator b are complete
//   ps_ready[b]  leader's; 256 arrivals: both epilogues have written their bf16 s*P rows to shared memory
//   acc_full[b]  per CTA; commit multicast: accumulator b incl. the rank-r product is complete
//   acc_empty[b] leader's; 256 arrivals: both epilogues have drained accumulator b
// Forward: the weight/adapter rows of a tile are K-major and contiguous, so ONE MMA of width block_n + r_pad
// gives the dense accumulator and P side by side (leader holds rows [0, half), peer the rest incl. A).
// Backward: W and A are MN-major operands in their natural layout (no transposed weight copy).  s (dY B)^T is
// computed beforehand by the skinny streaming kernel (narrow side MMAs in the main loop cost ~40 cycles each
// whatever their width), so the tile is a plain K-extended GEMM: after the d_out/64 main k-blocks one more
// k-block of depth r_pad multiplies the Qt tile (MN-major A operand, straight from TMA) with the rows of A.
#include "kernels.h"
#include "sm100_ptx.cuh"

namespace lora {

namespace {

// The 16 NF4 levels (QLoRA, Appendix E: normal quantiles scaled to [-1, 1] with an exact zero), float32.
__device__ __constant__ float c_nf4_levels[16] = {
    -1.0f, -0.6961928009986877f, -0.5250730514526367f, -0.39491748809814453f,
    -0.28444138169288635f, -0.18477343022823334f, -0.09105003625154495f, 0.0f,
    0.07958029955625534f, 0.16093020141124725f, 0.24611230194568634f, 0.33791524171829224f,
    0.44070982933044434f, 0.5626170039176941f, 0.7229568362236023f, 1.0f};

constexpr int kPairBarriers = kGemmBarriers + 2 * kNf4CodeSlots;   // + code ring full / empty (NF4 weight only)
constexpr int kPairBarrierBytes = 512;                             // barriers, TMEM slot, abort flag

struct PairTile {
  int m_idx, n_idx;
};

__device__ __forceinline__ PairTile pair_tile(int id, const GemmParams& p) {
  const int per_band = p.group_m * p.tiles_n;
  const int band = id / per_band;
  const int rem = id - band * per_band;
  const int rows = min(p.group_m, p.tiles_m - band * p.group_m);
  PairTile c;
  c.m_idx = band * p.group_m + rem % rows;
  c.n_idx = rem / rows;
  return c;
}

// kBmn: the weight-side operands (W, and A in the rank-r k-block) are MN-major (backward) instead of K-major.
// kExt: K-extended form - the scaled first adapter product (Pt or Qt, [r_pad, T] bf16) was computed beforehand and
//       enters as one more k-block; otherwise (forward only) it is fused: extra accumulator columns + epilogue.
//       With r_pad = 0 the K-extended form has no rank-r k-block at all: a plain GEMM.
// kAmn: the activation-side operand is MN-major too: its tensor is [K, M] row-major (box 64(m) x 64(k), two per stage).
//       This is the dense weight gradient dW = dY^T X, where both operands are contracted over their row index.
// kNf4: the frozen weight is held in 4-bit NormalFloat (Section 4.5, Q+LoRA).  Its packed codes and block scales are
//       staged by TMA into a small ring; four extra warps turn each 64-element block into bf16(level * absmax) and
//       write it into the stage's weight tile in exactly the swizzled layout TMA would have produced, so the MMA
//       side is unchanged.  K-extended form only (tm_w0 = codes, tm_w1 = absmax).
template <bool kBmn, bool kExt, bool kAmn = false, bool kNf4 = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kNf4 ? kPairThreadsNf4 : kPairThreads, 1)
lora_gemm_pair_kernel(const __grid_constant__ CUtensorMap tm_act,   // X / dY [M, K], box 64(k) x 128 ; kAmn: [K, M], box 64(m) x 64(k)
                      const __grid_constant__ CUtensorMap tm_w0,    // fwd: W box 64(k) x half ; bwd: W box 64(n) x 64(k)
                      const __grid_constant__ CUtensorMap tm_w1,    // fwd: W box 64(k) x (block_n - half) ; bwd unused
                      const __grid_constant__ CUtensorMap tm_side,  // fwd: A box 64(k) x r_pad ; bwd: Qt [r_pad, T] box 64(t) x r_pad
                      const __grid_constant__ CUtensorMap tm_tail,  // fwd: B box 64(r) x block_n/2 ; bwd: A box 64(n) x r_pad
                      const __grid_constant__ CUtensorMap tm_out,   // Y / dX [M, N], box 64 x 128
                      const GemmParams p) {
  constexpr int kStage = kPairStageBytesFwd;
  pdl_launch_dependents();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t ring = smem_u32(smem);
  const uint32_t staging = ring + p.stages * kStage;
  uint8_t* staging_ptr = smem + p.stages * kStage;
  uint64_t* bars = reinterpret_cast<uint64_t*>(staging_ptr + 2 * kStagingBytes);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
  auto side_full = [&](int b) { return bar0 + 8u * (2 * kMaxStages + b); };
  auto ps_ready = [&](int b) { return bar0 + 8u * (2 * kMaxStages + 2 + b); };
  auto acc_full = [&](int b) { return bar0 + 8u * (2 * kMaxStages + 4 + b); };
  auto acc_empty = [&](int b) { return bar0 + 8u * (2 * kMaxStages + 6 + b); };
  auto cfull_bar = [&](int c) { return bar0 + 8u * (kGemmBarriers + c); };
  auto cempty_bar = [&](int c) { return bar0 + 8u * (kGemmBarriers + kNf4CodeSlots + c); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kPairBarriers);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  // NF4 only: ring of packed codes + block scales, and the byte -> (level of low nibble, level of high nibble) table
  uint8_t* code_ring = staging_ptr + 2 * kStagingBytes + kPairBarrierBytes;
  // level table replicated once per lane: entry (code, lane) at word code * 32 + lane, so a warp's 32 lookups with
  // arbitrary codes hit 32 different banks (a shared 16- or 256-entry table serialises on bank conflicts and made the
  // shared-memory pipe the bottleneck)
  float* nf4_lut = reinterpret_cast<float*>(code_ring + kNf4CodeSlots * kNf4CodeSlotBytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_cta_rank();

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(full_bar(s), kNf4 ? 1 + 2 * kNf4WarpsPerGroup : 2);   // NF4: the dequantising warps of one group, both CTAs
      mbar_init(empty_bar(s), 1);
    }
    if (kNf4) {
      for (int c = 0; c < kNf4CodeSlots; ++c) {
        mbar_init(cfull_bar(c), 1);
        mbar_init(cempty_bar(c), kNf4WarpsPerGroup);
      }
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(side_full(b), 1);
      mbar_init(ps_ready(b), 256);
      mbar_init(acc_full(b), 1);
      mbar_init(acc_empty(b), 256);
    }
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tm_act);
    tma_prefetch_desc(&tm_w0);
    tma_prefetch_desc(&tm_w1);
    tma_prefetch_desc(&tm_side);
    tma_prefetch_desc(&tm_tail);
    tma_prefetch_desc(&tm_out);
  }
  if (warp == 4) {
    tmem_alloc_pair(smem_u32(tmem_slot), 512);
    tmem_relinquish_pair();
  }
  if (kNf4 && threadIdx.x >= kPairThreads) {
    for (int b = threadIdx.x - kPairThreads; b < 16 * 32; b += kNf4DequantThreads) nf4_lut[b] = c_nf4_levels[b >> 5];
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();           // the peer's barriers exist before anything is signalled across the pair
  tc_fence_after();
  pdl_wait();                   // everything above overlapped the previous kernel's tail; global memory from here on
  const uint32_t tmem_base = *tmem_slot;
  // one thread of the grid notes wall time and SM clock when its CTA starts working and when it leaves: the host derives
  // the SM frequency this launch really ran at (bytes 64..95 of the status block, see lora_plan_last_gemm_clock)
  unsigned long long t_begin = 0;
  long long c_begin = 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_begin));
    c_begin = clock64();
  }

  const int G = gridDim.x >> 1;                 // CTA pairs
  const int pair = blockIdx.x >> 1;
  // work items: (tile, k-split).  split_k > 1 only in the K-extended form: each item covers kb_per_split main k-blocks,
  // the last split also the rank-r k-block, and the epilogue writes an fp32 partial tile instead of bf16 output
  const int SK = kExt ? p.split_k : 1;
  const int n_items = p.num_tiles * SK;
  const int n_my = (n_items > pair) ? (n_items - 1 - pair) / G + 1 : 0;
  const int KB = p.kblocks;
  const int D = min(KB, p.tail_delay);
  const int S = p.stages;
  const int BN = p.block_n;
  const int half = (BN + p.r_pad) >> 1;         // forward: weight/adapter rows held by each CTA

  if (warp < 4) {
    // ================================ TMA producers (both CTAs) ================================
    // warp = 2 * parity + operand: operand 0 = activation tile, 1 = weight (+ adapter) tile; the warp handles the
    // ring items whose index has its parity.  Ring position, phase and tile coordinates are carried as counters
    // (no division in the loop); one lane polls, one elected lane issues.
    const int op = warp & 1, par = warp >> 1;
    int slot = 0, phase = 0, odd = 0;
    bool ok = true;
    // claims the next ring item; returns its slot or -1 when the item belongs to the other warp pair
    auto acquire = [&]() -> int {
      const int mine = (odd == par), cur = slot;
      if (mine) ok = warp_wait(empty_bar(cur), phase ^ 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_EMPTY, false, 20);
      if (++slot == S) { slot = 0; phase ^= 1; }
      odd ^= 1;
      return mine ? cur : -1;
    };
    auto load_main = [&](int m0, int n0, int k0) {
      const int cur = acquire();
      if (cur < 0 || !ok) return;
      const uint32_t a_dst = ring + cur * kStage, b_dst = a_dst + 16384;
      const uint32_t fb = map_to_cta(full_bar(cur), 0);
      if (elect_one()) {
        if (op == 0) {
          if (rank == 0) mbar_arrive_expect_tx(full_bar(cur), 2 * 16384);
          if (!kAmn) {
            tma_load_2d_pair(a_dst, &tm_act, fb, k0, m0);
          } else {
            tma_load_2d_pair(a_dst, &tm_act, fb, m0, k0);
            tma_load_2d_pair(a_dst + 8192, &tm_act, fb, m0 + 64, k0);
          }
        } else if (!kExt) {
          if (rank == 0) {
            mbar_arrive_expect_tx(full_bar(cur), (BN + p.r_pad) * 128);
            tma_load_2d_pair(b_dst, &tm_w0, fb, k0, n0);
          } else {
            tma_load_2d_pair(b_dst, &tm_w1, fb, k0, n0 + half);
            tma_load_2d_pair(b_dst + (BN - half) * 128, &tm_side, fb, k0, 0);
          }
        } else if (!kBmn) {
          if (rank == 0) mbar_arrive_expect_tx(full_bar(cur), BN * 128);
          tma_load_2d_pair(b_dst, &tm_w0, fb, k0, n0 + static_cast<int>(rank) * (BN >> 1));
        } else {
          if (rank == 0) mbar_arrive_expect_tx(full_bar(cur), 2 * 16384);
          const int nb = n0 + static_cast<int>(rank) * (BN >> 1);
          tma_load_2d_pair(b_dst, &tm_w0, fb, nb, k0);
          tma_load_2d_pair(b_dst + 8192, &tm_w0, fb, nb + 64, k0);
        }
      }
      __syncwarp();
    };
    // K-extended forms, grouped projections: the rank-r k-block of a FORWARD tile takes the rows of s (X A^T)^T that belong
    // to the tile's group (srow = group x r_pad, one part); the dX GEMM adds one part per group (rows part x r_pad of
    // s (dY B)^T and of the stacked A).  Ungrouped: one part, row 0.
    auto load_tail = [&](int m0, int n0, int part) {
      const int cur = acquire();
      if (cur < 0 || !ok) return;
      const int nb = n0 + static_cast<int>(rank) * (BN >> 1);
      int srow = part * p.r_pad;
      if (kExt && !kBmn && p.n_groups > 1) {
        int g = 0;
        while (g + 1 < p.n_groups && n0 >= p.group_end[g]) ++g;
        srow = g * p.r_pad;
      }
      const uint32_t a_dst = ring + cur * kStage, b_dst = a_dst + 16384;
      const uint32_t fb = map_to_cta(full_bar(cur), 0);
      if (elect_one()) {
        if (op == 0) {
          if (!kExt) {
            if (rank == 0) mbar_arrive(full_bar(cur));        // fused: the rank-r operand comes from the epilogue
          } else {
            // K-extended: s (X A^T)^T or s (dY B)^T for this CTA's 128 tokens, two 64-token groups of r_pad rows (MN-major A operand)
            // (NF4: this warp also brings the weight-side operand of the rank-r k-block; the other producer warps
            // only feed the code ring)
            const uint32_t side_bytes = 2 * 2 * p.r_pad * 128;
            const uint32_t tail_bytes = kNf4 ? (kBmn ? 2 * 2 * p.r_pad * 128 : BN * 128) : 0;
            if (rank == 0) mbar_arrive_expect_tx(full_bar(cur), side_bytes + tail_bytes);
            tma_load_2d_pair(a_dst, &tm_side, fb, m0, srow);
            tma_load_2d_pair(a_dst + p.r_pad * 128, &tm_side, fb, m0 + 64, srow);
            if (kNf4 && !kBmn) {
              tma_load_2d_pair(b_dst, &tm_tail, fb, 0, nb);
            } else if (kNf4) {
              tma_load_2d_pair(b_dst, &tm_tail, fb, nb, 0);
              tma_load_2d_pair(b_dst + 8192, &tm_tail, fb, nb + 64, 0);
            }
          }
        } else if (!kBmn) {
          if (rank == 0) mbar_arrive_expect_tx(full_bar(cur), BN * 128);
          tma_load_2d_pair(b_dst, &tm_tail, fb, 0, nb);
        } else {
          if (rank == 0) mbar_arrive_expect_tx(full_bar(cur), 2 * 2 * p.r_pad * 128);
          tma_load_2d_pair(b_dst, &tm_tail, fb, nb, srow);
          tma_load_2d_pair(b_dst + 8192, &tm_tail, fb, nb + 64, srow);
        }
      }
      __syncwarp();
    };
    if (kNf4 && op == 1) {
      // ---- NF4: these two warps feed the code ring (packed codes + block scales of every main k-block) ----
      int cslot = 0, cphase = 0, codd = 0;
      for (int i = 0; i < n_my && ok; ++i) {
        const int item = pair + i * G, sp = item % SK;
        const PairTile tc = pair_tile(item / SK, p);
        const int nb = tc.n_idx * BN + static_cast<int>(rank) * (BN >> 1);
        const int kb0 = sp * p.kb_per_split, kb1 = min(KB, kb0 + p.kb_per_split);
        for (int kb = kb0; kb < kb1 && ok; ++kb) {
          if (codd == par) {
            ok = warp_wait(cempty_bar(cslot), cphase ^ 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_EMPTY, false, 20);
            if (ok && elect_one()) {
              const uint32_t cdst = smem_u32(code_ring) + cslot * kNf4CodeSlotBytes, cb = cfull_bar(cslot);
              mbar_arrive_expect_tx(cb, kNf4CodeSlotBytes);
              if (!kBmn) {   // forward: rows nb.. of W, the 32 code bytes and the one scale of k-block kb
                tma_load_2d(cdst, &tm_w0, cb, kb * 32, nb);
                tma_load_2d(cdst + 4096, &tm_w1, cb, nb, kb);
              } else {       // backward: rows kb*64.. of W (the contraction index), 128 columns = 64 code bytes, 2 blocks
                tma_load_2d(cdst, &tm_w0, cb, nb >> 1, kb * kBlockK);
                tma_load_2d(cdst + 4096, &tm_w1, cb, kb * kBlockK, nb >> 6);
              }
            }
            __syncwarp();
          }
          if (++cslot == kNf4CodeSlots) { cslot = 0; cphase ^= 1; }
          codd ^= 1;
        }
      }
    }
    // Item order.  Fused: the rank-r item of tile i-1 comes D k-blocks into tile i (its operand is made by the
    // epilogue meanwhile).  K-extended: the rank-r item is simply the last k-block of its own tile.
    int prev_n0 = 0;
    for (int i = 0; i < n_my && ok && !(kNf4 && op == 1); ++i) {
      const int item = pair + i * G, sp = item % SK;
      const PairTile tc = pair_tile(item / SK, p);
      const int m0 = tc.m_idx * kPairBlockM + static_cast<int>(rank) * 128, n0 = tc.n_idx * BN;
      const int kb0 = sp * p.kb_per_split, kb1 = min(KB, kb0 + p.kb_per_split);
      for (int kb = kb0; kb < kb1 && ok; ++kb) {
        if (!kExt && i > 0 && kb == D) load_tail(0, prev_n0, 0);
        if (ok) load_main(m0, n0, kb * kBlockK);
      }
      if (!kExt && ok && i > 0 && D == KB) load_tail(0, prev_n0, 0);
      if (kExt && sp == SK - 1 && p.r_pad > 0)
        for (int part = 0; part < p.tail_parts && ok; ++part) load_tail(m0, n0, part);
      prev_n0 = n0;
    }
    if (!kExt && ok && n_my > 0 && !(kNf4 && op == 1)) load_tail(0, prev_n0, 0);
  } else if (warp == 4) {
    // ================================ MMA issuer (leader CTA only) ================================
    // Whole warp of the leader CTA runs the loop; one lane polls, one elected lane issues every MMA and commit.
    // Descriptors are advanced by adding byte offsets (>> 4) to precomputed bases.
    if (rank == 0) {
      const uint32_t idesc_main = kExt ? mma_idesc_bf16(256, BN, kAmn, kBmn) : mma_idesc_bf16(256, BN + p.r_pad, false, false);
      const uint32_t idesc_tail = mma_idesc_bf16(256, BN, kExt, kBmn);   // K-extended: Pt / Qt is an MN-major A operand
      const uint64_t ad0 = kAmn ? smem_desc_sw128(ring, 8192, 1024) : smem_desc_sw128(ring, 16, 1024);
      constexpr uint32_t kAStep = kAmn ? (2048 >> 4) : (32 >> 4);
      const uint64_t bd0 = kBmn ? smem_desc_sw128(ring + 16384, 8192, 1024) : smem_desc_sw128(ring + 16384, 16, 1024);
      // rank-r A operand: forward = bf16 s*P rows written by the epilogue (K-major, in the staging buffer);
      // backward = Qt tile delivered by TMA into the stage's activation part (MN-major, two 64-token groups)
      const uint64_t pd0 = kExt ? smem_desc_sw128(ring, p.r_pad * 128, 1024) : smem_desc_sw128(staging, 16, 1024);
      constexpr uint32_t kPStep = kExt ? (2048 >> 4) : (32 >> 4);
      constexpr uint32_t kBStep = kBmn ? (2048 >> 4) : (32 >> 4);     // descriptor step per 16-wide k-step
      int slot = 0, phase = 0;
      bool ok = true;
      auto next = [&]() { if (++slot == S) { slot = 0; phase ^= 1; } };
      auto mma_main = [&](int buf, bool first_kb, bool last_kb, bool has_tail) {
        ok = warp_wait(full_bar(slot), phase, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_FULL, true, 0);
        if (!ok) return;
        tc_fence_after();
        if (elect_one()) {
          const uint32_t so = static_cast<uint32_t>(slot * kStage) >> 4;
          const uint32_t acc = tmem_base + buf * 256;
#pragma unroll
          for (int ks = 0; ks < kBlockK / 16; ++ks) {
            const uint32_t accum = (!first_kb || ks != 0) ? 1u : 0u;
            const uint64_t ad = ad0 + so + ks * kAStep;
            mma_bf16_ss_pair(acc, ad, bd0 + so + ks * kBStep, idesc_main, accum);
          }
          mma_commit_pair(empty_bar(slot));
          if (!kExt && last_kb) mma_commit_pair(side_full(buf));
          if (kExt && last_kb && !has_tail) mma_commit_pair(acc_full(buf));
        }
        __syncwarp();
        next();
      };
      auto mma_tail = [&](int buf, int use, bool last_part) {
        if (!kExt) ok = warp_wait(ps_ready(buf), use & 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_PS, true, 0);
        if (ok) ok = warp_wait(full_bar(slot), phase, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_FULL, true, 0);
        if (!ok) return;
        tc_fence_after();
        if (elect_one()) {
          const uint32_t so = static_cast<uint32_t>(slot * kStage) >> 4;
          for (int ks = 0; ks < p.r_pad / 16; ++ks)
            mma_bf16_ss_pair(tmem_base + buf * 256, pd0 + (kExt ? so : 0u) + ks * kPStep, bd0 + so + ks * kBStep, idesc_tail, 1u);
          mma_commit_pair(empty_bar(slot));
          if (last_part) mma_commit_pair(acc_full(buf));
        }
        __syncwarp();
        next();
      };
      for (int i = 0; i < n_my && ok; ++i) {
        const int buf = i & 1, use = i >> 1;
        const int sp = (pair + i * G) % SK;
        const int kb0 = sp * p.kb_per_split, kb1 = min(KB, kb0 + p.kb_per_split);
        const bool has_tail = !kExt || (sp == SK - 1 && p.r_pad > 0);
        ok = warp_wait(acc_empty(buf), (use & 1) ^ 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_ACC_EMPTY, true, 0);
        for (int kb = kb0; kb < kb1 && ok; ++kb) {
          if (!kExt && i > 0 && kb == D) mma_tail(buf ^ 1, (i - 1) >> 1, true);
          if (ok) mma_main(buf, kb == kb0, kb == kb1 - 1, has_tail);
        }
        if (!kExt && ok && i > 0 && D == KB) mma_tail(buf ^ 1, (i - 1) >> 1, true);
        if (kExt && has_tail)
          for (int part = 0; part < p.tail_parts && ok; ++part) mma_tail(buf, use, part == p.tail_parts - 1);
      }
      if (!kExt && ok && n_my > 0) mma_tail((n_my - 1) & 1, (n_my - 1) >> 1, true);
    }
  } else if (kNf4 && warp >= kPairThreads / 32) {
    // ================================ NF4 dequantisation (warps 9..16, 256 threads per CTA) ================================
    // The eight warps form kNf4Groups groups of kNf4WarpsPerGroup warps; ring items go to the groups round-robin, so
    // several items are converted at once.  One item's conversion is a long dependent chain (wait, code fetch, table
    // look-ups, stores, proxy fence: measured ~3000 cycles when all warps shared each item) while the tensor core
    // consumes an item in ~512 cycles; only concurrency across items hides that chain.
    // A group's 64 threads own the 128 quantisation blocks of an item, two each (32 code bytes + one scale in, 128 bytes
    // of bf16 out per block):
    //   forward  (weight rows K-major):  block u = row u of this CTA's weight rows, the k-block's 64 input features
    //   backward (weight MN-major):      block u = contraction row u % 64 of the k-block, column group u / 64
    // Every element is bf16(level * absmax): one float32 product, one round-to-nearest-even.
    const int dwarp = warp - kPairThreads / 32;
    const int gid = dwarp / kNf4WarpsPerGroup;
    const int t = (dwarp % kNf4WarpsPerGroup) * 32 + lane;
    const uint32_t lut_lane = smem_u32(nf4_lut) + 4u * lane;
    const uint32_t code_ring_u32 = smem_u32(code_ring);
    int slot = 0, phase = 0, cslot = 0, cphase = 0, turn = 0;
    bool ok = true;
    for (int i = 0; i < n_my && ok; ++i) {
      const int sp = (pair + i * G) % SK;
      const int kb0 = sp * p.kb_per_split, kb1 = min(KB, kb0 + p.kb_per_split);
      const bool has_tail = sp == SK - 1 && p.r_pad > 0;
      for (int kb = kb0; kb < kb1 + (has_tail ? p.tail_parts : 0) && ok; ++kb) {
        const bool main_item = kb < kb1;
        if (turn == gid) {
          if (main_item) ok = warp_wait(cfull_bar(cslot), cphase, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_FULL, false, 0);
          if (ok) ok = warp_wait(empty_bar(slot), phase ^ 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_EMPTY, false, 0);
          if (!ok) break;
          if (main_item) {
            (void)mbar_try_wait(cfull_bar(cslot), cphase);     // every reading thread observes the completed copy itself
            const uint32_t src = code_ring_u32 + cslot * kNf4CodeSlotBytes;
            const uint32_t stage_b = ring + slot * kStage + 16384;
#pragma unroll
            for (int h = 0; h < 128 / (32 * kNf4WarpsPerGroup); ++h) {
              const int u = t + h * 32 * kNf4WarpsPerGroup;
              const int row = kBmn ? (u & 63) : u;
              const int grp = kBmn ? (u >> 6) : 0;
              if (!kBmn && u >= (BN >> 1)) continue;           // forward: this CTA holds block_n / 2 weight rows
              const uint32_t code_addr = src + (kBmn ? static_cast<uint32_t>(row * 64 + grp * 32) : static_cast<uint32_t>(row * 32));
              const uint4 c0 = lds_v4(code_addr), c1 = lds_v4(code_addr + 16);
              const float scale = lds_f32(src + 4096u + 4u * static_cast<uint32_t>(u));
              const uint32_t dst = stage_b + grp * 8192;
              const uint32_t cw[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
              for (int q = 0; q < 8; ++q) {     // 4 code bytes -> 8 elements -> one 16-byte chunk of the swizzled row
                uint32_t w[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const float lo = lds_const_f32(lut_lane + (((cw[q] >> (8 * j)) & 0xFu) << 7));
                  const float hi = lds_const_f32(lut_lane + (((cw[q] >> (8 * j + 4)) & 0xFu) << 7));
                  w[j] = pack_bf16x2(lo * scale, hi * scale);
                }
                sts_v4(dst + sw128_offset(row, q), w[0], w[1], w[2], w[3]);
              }
            }
            fence_proxy_async_smem();           // the tensor core reads the tile through the async proxy
          }
          // one arrival per warp: every lane's writes and fence come before the warp barrier, the elected lane's
          // release-arrive after it
          __syncwarp();
          if (lane == 0) {
            if (main_item) mbar_arrive(cempty_bar(cslot));
            mbar_arrive_cluster(map_to_cta(full_bar(slot), 0));
          }
        }
        if (++turn == kNf4Groups) turn = 0;
        if (main_item && ++cslot == kNf4CodeSlots) { cslot = 0; cphase ^= 1; }
        if (++slot == S) { slot = 0; phase ^= 1; }
      }
    }
  } else {
    // ================================ epilogue (128 threads per CTA) ================================
    const int e = threadIdx.x - 160;
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    const int full_chunks = BN >> 6;
    const int rem_cols = BN & 63;                  // 0, 16, 32 or 48 columns stored with plain stores
    for (int i = 0; i < n_my; ++i) {
      const int item = pair + i * G, sp = item % SK;
      const PairTile tc = pair_tile(item / SK, p);
      const int m0 = tc.m_idx * kPairBlockM + static_cast<int>(rank) * 128, n0 = tc.n_idx * BN;
      const int buf = i & 1, use = i >> 1;
      bool ok = true;
      if (e == 0) tma_store_wait_read<0>();       // the previous tile's stores have left both staging buffers
      if (!kExt) {
        // ---- fused forward: P = X A^T from TMEM -> scale -> bf16 -> shared memory as the rank-r MMA operand ----
        ok = warp_wait(side_full(buf), use & 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_SIDE, false, 64);
        if (named_bar_or(1, 128, !ok)) break;
        tc_fence_after();
        for (int c16 = 0; c16 < p.r_pad / 16; ++c16) {
          uint32_t v[16];
          tmem_ld16(lane_addr + buf * 256 + BN + c16 * 16, v);
          tmem_ld_wait();
          uint32_t w[8];
#pragma unroll
          for (int q = 0; q < 8; ++q)
            w[q] = pack_bf16x2(__uint_as_float(v[2 * q]) * p.scale, __uint_as_float(v[2 * q + 1]) * p.scale);
          *reinterpret_cast<uint4*>(staging_ptr + sw128_offset(row, 2 * c16)) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(staging_ptr + sw128_offset(row, 2 * c16 + 1)) = make_uint4(w[4], w[5], w[6], w[7]);
          if (p.rt_out != nullptr && tc.n_idx == 0 && m0 + row < p.M) {
            // keep s (X A^T)^T for a backward pass that reuses it
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
        mbar_arrive_cluster(map_to_cta(ps_ready(buf), 0));
      }
      ok = warp_wait(acc_full(buf), use & 1, abort_flag, p.status, p.wait_limit, DEV_TIMEOUT_ACC, false, 32);
      if (named_bar_or(1, 128, !ok)) break;
      tc_fence_after();
      if (kExt && SK > 1) {
        // ---- split along K: this item's fp32 partial tile -> part[sp][row][col], 16 columns at a time ----
        float* prow = p.part + (static_cast<size_t>(sp) * p.M + (m0 + row)) * p.N;
        for (int c16 = 0; c16 < BN / 16; ++c16) {
          uint32_t v[16];
          tmem_ld16(lane_addr + buf * 256 + c16 * 16, v);
          tmem_ld_wait();
          if (c16 == BN / 16 - 1) {
            tc_fence_before();
            mbar_arrive_cluster(map_to_cta(acc_empty(buf), 0));
          }
          const int col = n0 + c16 * 16;
          if (m0 + row < p.M) {
#pragma unroll
            for (int q = 0; q < 4; ++q)
              if (col + 4 * q < p.N)
                *reinterpret_cast<uint4*>(prow + col + 4 * q) = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
          }
        }
        continue;
      }
      for (int c = 0; c < full_chunks; ++c) {
        uint32_t v0[32], v1[32];
        tmem_ld32(lane_addr + buf * 256 + c * 64, v0);
        tmem_ld32(lane_addr + buf * 256 + c * 64 + 32, v1);
        tmem_ld_wait();
        if (c == full_chunks - 1 && rem_cols == 0) {
          tc_fence_before();
          mbar_arrive_cluster(map_to_cta(acc_empty(buf), 0));
        }
        if (n0 + c * 64 >= p.N) continue;
        if (e == 0) tma_store_wait_read<1>();
        named_bar_sync(2, 128);
        uint8_t* dst = staging_ptr + (c & 1) * kStagingBytes;
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
      if (rem_cols != 0) {
        // ragged last chunk (block_n is not a multiple of 64): 16 columns at a time, plain 16-byte stores
        const int cbase = full_chunks * 64;
        for (int c16 = 0; c16 < rem_cols / 16; ++c16) {
          uint32_t v[16];
          tmem_ld16(lane_addr + buf * 256 + cbase + c16 * 16, v);
          tmem_ld_wait();
          if (c16 == rem_cols / 16 - 1) {
            tc_fence_before();
            mbar_arrive_cluster(map_to_cta(acc_empty(buf), 0));
          }
          const int col = n0 + cbase + c16 * 16;
          if (m0 + row < p.M) {
            uint4 w0, w1;
            w0.x = pack_bf16x2(__uint_as_float(v[0]), __uint_as_float(v[1]));
            w0.y = pack_bf16x2(__uint_as_float(v[2]), __uint_as_float(v[3]));
            w0.z = pack_bf16x2(__uint_as_float(v[4]), __uint_as_float(v[5]));
            w0.w = pack_bf16x2(__uint_as_float(v[6]), __uint_as_float(v[7]));
            w1.x = pack_bf16x2(__uint_as_float(v[8]), __uint_as_float(v[9]));
            w1.y = pack_bf16x2(__uint_as_float(v[10]), __uint_as_float(v[11]));
            w1.z = pack_bf16x2(__uint_as_float(v[12]), __uint_as_float(v[13]));
            w1.w = pack_bf16x2(__uint_as_float(v[14]), __uint_as_float(v[15]));
            __nv_bfloat16* orow = p.out + static_cast<size_t>(m0 + row) * p.ld_out;
            if (col < p.N) *reinterpret_cast<uint4*>(orow + col) = w0;
            if (col + 8 < p.N) *reinterpret_cast<uint4*>(orow + col + 8) = w1;
          }
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
  cluster_sync_all();                        // neither CTA leaves while the other may still touch its memory
  if (warp == 4) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 512);
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    unsigned long long t_end;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_end));
    unsigned long long* rec = reinterpret_cast<unsigned long long*>(p.status) + 8;
    rec[0] = t_begin;
    rec[1] = t_end;
    rec[2] = static_cast<unsigned long long>(c_begin);
    rec[3] = static_cast<unsigned long long>(clock64());
  }
}

// out[t, n] = bf16( sum over k-splits of part[sp][t][n] ), splits added in index order; 8 outputs per thread
__global__ void __launch_bounds__(256) lora_splitk_reduce_kernel(const float* part, __nv_bfloat16* out, long long n_elems,
                                                                int splits) {
  pdl_launch_dependents();
  pdl_wait();
  const long long i = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) * 8;
  if (i >= n_elems) return;
  float acc[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) acc[q] = 0.f;
  for (int s = 0; s < splits; ++s) {
    const float4 a = __ldcg(reinterpret_cast<const float4*>(part + s * n_elems + i));
    const float4 b = __ldcg(reinterpret_cast<const float4*>(part + s * n_elems + i + 4));
    acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w;
    acc[4] += b.x; acc[5] += b.y; acc[6] += b.z; acc[7] += b.w;
  }
  uint4 w;
  w.x = pack_bf16x2(acc[0], acc[1]);
  w.y = pack_bf16x2(acc[2], acc[3]);
  w.z = pack_bf16x2(acc[4], acc[5]);
  w.w = pack_bf16x2(acc[6], acc[7]);
  *reinterpret_cast<uint4*>(out + i) = w;
}

}  // namespace

cudaError_t launch_splitk_reduce(const float* part, __nv_bfloat16* out, long long n_elems, int splits, cudaStream_t stream) {
  const long long threads = (n_elems + 7) / 8;
  return launch_pdl(lora_splitk_reduce_kernel, dim3(static_cast<unsigned>((threads + 255) / 256)), dim3(256), 0, stream, part,
                    out, n_elems, splits);
}

size_t gemm_pair_smem_bytes(int stages, bool nf4) {
  return static_cast<size_t>(stages) * kPairStageBytesFwd + 2 * kStagingBytes + kPairBarrierBytes + 1024 +
         (nf4 ? kNf4CodeSlots * kNf4CodeSlotBytes + 16 * 32 * sizeof(float) : 0);
}

cudaError_t gemm_pair_configure() {
  cudaError_t e = cudaFuncSetAttribute(lora_gemm_pair_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(lora_gemm_pair_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(lora_gemm_pair_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(lora_gemm_pair_kernel<true, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(lora_gemm_pair_kernel<false, true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(lora_gemm_pair_kernel<true, true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
  return e;
}

cudaError_t launch_gemm_pair_fwd(const CUtensorMap& tmX, const CUtensorMap& tmW0, const CUtensorMap& tmW1,
                                 const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmY,
                                 const GemmParams& p, int ctas, cudaStream_t stream) {
  return launch_pdl(lora_gemm_pair_kernel<false, false>, dim3(ctas), dim3(kPairThreads), gemm_pair_smem_bytes(p.stages, false), stream,
                    tmX, tmW0, tmW1, tmA, tmB, tmY, p);
}

cudaError_t launch_gemm_pair_fwd_ext(const CUtensorMap& tmX, const CUtensorMap& tmW, const CUtensorMap& tmPt,
                                     const CUtensorMap& tmB, const CUtensorMap& tmY, const GemmParams& p, int ctas,
                                     cudaStream_t stream) {
  return launch_pdl(lora_gemm_pair_kernel<false, true>, dim3(ctas), dim3(kPairThreads), gemm_pair_smem_bytes(p.stages, false), stream,
                    tmX, tmW, tmW, tmPt, tmB, tmY, p);
}

cudaError_t launch_gemm_pair_dx(const CUtensorMap& tmdY, const CUtensorMap& tmW, const CUtensorMap& tmQt,
                                const CUtensorMap& tmA, const CUtensorMap& tmdX, const GemmParams& p, int ctas,
                                cudaStream_t stream) {
  return launch_pdl(lora_gemm_pair_kernel<true, true>, dim3(ctas), dim3(kPairThreads), gemm_pair_smem_bytes(p.stages, false), stream,
                    tmdY, tmW, tmW, tmQt, tmA, tmdX, p);
}

cudaError_t launch_gemm_pair_fwd_nf4(const CUtensorMap& tmX, const CUtensorMap& tmCodes, const CUtensorMap& tmAbsmax,
                                     const CUtensorMap& tmPt, const CUtensorMap& tmB, const CUtensorMap& tmY,
                                     const GemmParams& p, int ctas, cudaStream_t stream) {
  return launch_pdl(lora_gemm_pair_kernel<false, true, false, true>, dim3(ctas), dim3(kPairThreadsNf4),
                    gemm_pair_smem_bytes(p.stages, true), stream, tmX, tmCodes, tmAbsmax, tmPt, tmB, tmY, p);
}

cudaError_t launch_gemm_pair_dx_nf4(const CUtensorMap& tmdY, const CUtensorMap& tmCodes, const CUtensorMap& tmAbsmax,
                                    const CUtensorMap& tmQt, const CUtensorMap& tmA, const CUtensorMap& tmdX,
                                    const GemmParams& p, int ctas, cudaStream_t stream) {
  return launch_pdl(lora_gemm_pair_kernel<true, true, false, true>, dim3(ctas), dim3(kPairThreadsNf4),
                    gemm_pair_smem_bytes(p.stages, true), stream, tmdY, tmCodes, tmAbsmax, tmQt, tmA, tmdX, p);
}

cudaError_t launch_gemm_pair_dw(const CUtensorMap& tmdYt, const CUtensorMap& tmX, const CUtensorMap& tmdW, const GemmParams& p,
                                int ctas, cudaStream_t stream) {
  return launch_pdl(lora_gemm_pair_kernel<true, true, true>, dim3(ctas), dim3(kPairThreads), gemm_pair_smem_bytes(p.stages, false),
                    stream, tmdYt, tmX, tmX, tmX, tmX, tmdW, p);
}

}  // namespace lora
