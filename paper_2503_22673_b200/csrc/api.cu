// C ABI of the LoRA projection layer: argument checks, the per-shape selector, plans, tensor maps and
// kernel launches.  See include/lora_linear.h for the contract of every entry point.
#include "../../include/lora_linear.h"

#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "kernels.h"

namespace {

using namespace lora;

std::atomic<long long> g_launches{0};

constexpr size_t kAlign = 256;
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int ceil_div(long long a, long long b) { return static_cast<int>((a + b - 1) / b); }

// ------------------------------------------------------------------------------------------------
// selector
// ------------------------------------------------------------------------------------------------
// Cost model of one GEMM tile per 16-wide k-step, in SM cycles: the tensor pipe needs N_total / 2 cycles
// (128 x N_total x 16 MACs at 4096 MAC/cycle), the operand fetch from shared memory (128 + N_total) rows
// x 32 B at 128 B/cycle.  The tile width with the lowest (waves x per-tile cost) wins; wide tiles win on
// large grids, narrow tiles when the grid cannot fill the SMs.
int pick_block_n(long long T, long long N, int r_pad, int num_sms) {
  const int cands[3] = {192, 128, 64};
  int best = 192;
  double best_cost = 1e300;
  for (int bn : cands) {
    const long long tiles = static_cast<long long>(ceil_div(T, kBlockM)) * ceil_div(N, bn);
    const long long waves = (tiles + num_sms - 1) / num_sms;
    const double ntot = bn + r_pad;
    const double per_tile = (ntot / 2.0 > (128.0 + ntot) / 4.0) ? ntot / 2.0 : (128.0 + ntot) / 4.0;
    // fixed per-tile cost (rank-r MMA, accumulator hand-over), in the same unit, for a K of ~4096
    const double cost = static_cast<double>(waves) * (per_tile + 4.0);
    if (cost < best_cost - 1e-9) {
      best_cost = cost;
      best = bn;
    }
  }
  return best;
}

// CTA-pair tiles (256 rows): block_n is any multiple of 16 with block_n + r_pad <= 256.  Cost per tile is its
// MMA width (block_n + r_pad columns, the adapter columns ride along) plus a fixed hand-over cost; the
// width with the fewest (waves x cost) wins, ties go to the wider tile.
int pick_pair_block_n(long long T, long long N, int r_pad, int num_pairs) {
  if (const char* f = std::getenv("LORA_FORCE_BLOCK_N")) {
    const int v = std::atoi(f);
    if (v >= 64 && v % 16 == 0 && v + r_pad <= 256) return v;
  }
  if (r_pad == 0) {
    // K-extended GEMMs (no adapter columns; weight-side operand mostly MN-major).  Measured on dW 8192 x 4096 x 4096, us per
    // launch by width: 128: 262, 160: 236, 192: 201, 208: 240, 224: 209, 240: 219, 256: 184 - a wave costs 38-40 us up to
    // 192 columns (the 256-row activation tile is fetched per k-block whatever the width) and 46 us at 256, and widths
    // that are not multiples of 64 pay plain stores for their ragged last chunk.  So: 256 whenever that still gives
    // three quarters of the CTA pairs a tile; starved grids go through the width search below (narrower tiles buy parallelism there).
    const long long tiles256 = static_cast<long long>(ceil_div(T, kPairBlockM)) * ceil_div(N, 256);
    if (tiles256 * 4 >= static_cast<long long>(num_pairs) * 3) return 256;   // one 256-wide wave (46 us) beats one 240-wide (55 us)
  }
  int best = 256 - r_pad;
  double best_cost = 1e300;
  const int lo = r_pad + 32 > 144 ? r_pad + 32 : 144;
  for (int bn = 256 - r_pad; bn >= lo; bn -= 16) {
    const long long tiles = static_cast<long long>(ceil_div(T, kPairBlockM)) * ceil_div(N, bn);
    const long long waves = (tiles + num_pairs - 1) / num_pairs;
    const double cost = static_cast<double>(waves) * (bn + r_pad + 48.0);   // +48: accumulator hand-over, rank-r MMA, ramp
    if (cost < best_cost - 1e-9) {
      best_cost = cost;
      best = bn;
    }
  }
  return best;
}

// Streams of at most this many bytes run on a grid without cross-CTA sums (one launch instead of two): the whole
// problem is a few microseconds of work and the second launch would cost more than the parallelism gains.
constexpr long long kTinyStreamBytes = 1 << 20;

struct GradGrid {
  int feat_chunk, n_feat, n_tok, stages;
};

GradGrid pick_grad_grid(long long T, long long C, int r_pad, bool with_p, int num_sms) {
  GradGrid g;
  // TMEM: (feat_chunk / 128) accumulator blocks of r_pad columns + two r_pad-column buffers for X A^T <= 512
  int fc = (r_pad <= 32) ? 512 : 768;
  const int c128 = ceil_div(C, 128) * 128;
  if (fc > c128) fc = c128;
  g.feat_chunk = fc;
  g.n_feat = ceil_div(C, fc);
  const int n_slabs = ceil_div(T, kGradSlab);
  int n_tok = num_sms / g.n_feat;             // at most one CTA per SM: a second wave would double the time
  if (n_tok > n_slabs) n_tok = n_slabs;
  if (n_tok < 1) n_tok = 1;
  // tiny stream: one token chunk, so that no finalize launch is needed (pays only if the side product, where there is
  // one, needs no cross-CTA sum either)
  if (kTinyStreamBytes >= 2 * T * C && (!with_p || g.n_feat == 1)) n_tok = 1;
  g.n_tok = n_tok;
  const size_t stage = kGradStageBytes + (with_p ? 2 * static_cast<size_t>(r_pad) * 128 : 0);
  const size_t fixed = 4 * static_cast<size_t>(r_pad) * 128 + 2048;
  int stages = static_cast<int>((232448 - fixed) / stage);
  if (stages > kGradMaxStages) stages = kGradMaxStages;
  if (stages < 2) stages = 2;
  g.stages = stages;
  return g;
}

// Grid of a side-product-only pass (X A^T or dY B): feature chunks x token chunks.  No TMEM bound on the feature chunk.
//  * as few feature chunks (at most 4) as fill the SMs together with the 128-token slabs;
//  * ONE feature chunk for tiny streams and from 64 token slabs (8192 tokens) on: every CTA then sees all features, the
//    kernel writes the bf16 result itself and the finalize launch goes away (pre-pass stage 31.1 -> 30.7 us at
//    8192 x 4096, 107.9 -> 100.0 us at 16384 x 14336, one launch fewer each).
struct SideGrid {
  int feat_chunk, n_feat, n_tok;
};

SideGrid pick_side_grid(long long T, long long C, int num_sms) {
  const int n_slabs = ceil_div(T, kGradSlab);
  int nf = ceil_div(num_sms, n_slabs);
  if (nf > 4) nf = 4;
  if (kTinyStreamBytes >= 2 * T * C || n_slabs >= 64) nf = 1;
  if (const char* f = std::getenv("LORA_PREPASS_NF")) {      // tuning knob
    const int v = std::atoi(f);
    if (v >= 1 && v <= 4) nf = v;
  }
  SideGrid g;
  g.feat_chunk = ceil_div(ceil_div(C, nf), 128) * 128;
  g.n_feat = ceil_div(C, g.feat_chunk);
  g.n_tok = num_sms / g.n_feat;
  if (g.n_tok > n_slabs) g.n_tok = n_slabs;
  if (g.n_tok < 1) g.n_tok = 1;
  return g;
}

int check_shape(const lora_shape_t* s) {
  if (s == nullptr) return LORA_ERR_INVALID_ARG;
  if (s->T < 0 || s->d_in <= 0 || s->d_out <= 0 || s->r <= 0) return LORA_ERR_INVALID_ARG;
  if (s->T > (1ll << 30) || s->d_in > (1ll << 24) || s->d_out > (1ll << 24)) return LORA_ERR_UNSUPPORTED_SHAPE;
  if (s->d_in % 8 != 0 || s->d_out % 8 != 0) return LORA_ERR_UNSUPPORTED_SHAPE;
  if (s->r % 8 != 0 || s->r < 8 || s->r > 64) return LORA_ERR_UNSUPPORTED_SHAPE;
  return LORA_OK;
}

int select_config(const lora_shape_t* s, int num_sms, lora_kernel_config_t* c) {
  const int rc = check_shape(s);
  if (rc != LORA_OK) return rc;
  if (num_sms <= 0 || c == nullptr) return LORA_ERR_INVALID_ARG;
  std::memset(c, 0, sizeof(*c));
  const long long T = s->T > 0 ? s->T : 1;
  c->block_m = kBlockM;
  c->block_k = kBlockK;
  c->r_pad = static_cast<int>((s->r + 15) / 16 * 16);
  c->fwd_block_n = pick_block_n(T, s->d_out, c->r_pad, num_sms);
  c->dx_block_n = pick_block_n(T, s->d_in, c->r_pad, num_sms);
  c->stages = 4;
  c->dx_stages = 4;
  c->group_m = 8;
  if (const char* f = std::getenv("LORA_FORCE_GROUP_M")) {   // tuning knob: m-tiles per rasterisation band
    const int v = std::atoi(f);
    if (v >= 1 && v <= 64) c->group_m = v;
  }
  c->split_k = 1;
  c->dx_split_k = 1;
  c->tail_delay = 8;
  c->prefetch_dist = 0;    // L2 prefetch ahead of the ring was measured slower (it competes with the producers' copies)
  c->cta_group = (T > kBlockM && num_sms >= 2) ? 2 : 1;
  if (const char* f = std::getenv("LORA_FORCE_CTA_GROUP")) {
    const int v = std::atoi(f);
    if (v == 1 || (v == 2 && num_sms >= 2)) c->cta_group = v;
  }
  if (c->cta_group == 2) {
    const int pairs = num_sms / 2;
    c->block_m = kPairBlockM;
    c->fwd_block_n = pick_pair_block_n(T, s->d_out, c->r_pad, pairs);
    c->dx_block_n = pick_pair_block_n(T, s->d_in, 0, pairs);      // no adapter columns in the K-extended dX GEMM
    // Forward, fused vs K-extended.  Fused adapter columns cost r_pad / 256 of every MMA (time ~ T d_in d_out r_pad);
    // the alternative is a skinny X A^T pre-pass (time ~ T d_in, one more read of X) and 256-wide tiles.  Their ratio
    // is ~1e-5 d_out r_pad at the measured rates (1.2 PFLOP/s GEMM, 3 TB/s pre-pass), so the pre-pass wins for wide
    // outputs or large ranks.  Measured break-even: 4096 x 16 (fused 0.984 ms vs 0.926 ms K-extended at T = 32768 under
    // the power cap, where the wasted adapter columns also cost clock; 0.473 vs 0.456 ms per step at T = 8192), while
    // 1024 x 16 is faster fused (0.280 vs 0.291 ms): 14336 x 16, 4096 x 64 and 4096 x 16 take the pre-pass.
    // (between 65536 and 1e5 only from 4096 tokens on: below that the two extra launches weigh more than the columns)
    const long long dr = static_cast<long long>(s->d_out) * c->r_pad;
    c->fwd_ext = (dr >= 100000 || (dr >= 65536 && T >= 4096)) ? 1 : 0;
    if (const char* f = std::getenv("LORA_FORCE_FWD_EXT")) c->fwd_ext = std::atoi(f) != 0 ? 1 : 0;
    // Split along K: when the tiling leaves at least three quarters of the CTA pairs idle and the contraction is long
    // (>= 64 k-blocks), each tile is cut into k-ranges handled by different pairs (fp32 partial tiles, fixed-order
    // reduce kernel).  Measured: 257 x 14336 -> 264 forward 86 -> 45 us with 8 splits; on shorter contractions or
    // fuller grids (256 x 4096 x 4096: 29 tiles) the extra reduce launch costs as much as the split saves.
    // Only the K-extended kernel form supports it, so such a forward is K-extended too.
    auto pick_split = [&](long long tiles, int kb) {
      if (tiles * 4 > pairs || kb < 64) return 1;
      long long sp = pairs / tiles;
      if (sp > kb / 16) sp = kb / 16;
      if (sp > 8) sp = 8;
      return static_cast<int>(sp < 1 ? 1 : sp);
    };
    {
      const int bn = pick_pair_block_n(T, s->d_out, 0, pairs);
      const long long tiles = static_cast<long long>(ceil_div(T, kPairBlockM)) * ceil_div(s->d_out, bn);
      c->split_k = pick_split(tiles, ceil_div(s->d_in, kBlockK));
      if (c->split_k > 1) c->fwd_ext = 1;
    }
    if (c->fwd_ext) c->fwd_block_n = pick_pair_block_n(T, s->d_out, 0, pairs);
    {
      const long long tiles = static_cast<long long>(ceil_div(T, kPairBlockM)) * ceil_div(s->d_in, c->dx_block_n);
      c->dx_split_k = pick_split(tiles, ceil_div(s->d_out, kBlockK));
    }
    if (const char* f = std::getenv("LORA_FORCE_SPLIT_K")) {
      const int v = std::atoi(f);
      if (v >= 1 && v <= 8) {
        c->split_k = c->dx_split_k = v;
        if (v > 1 && !c->fwd_ext) { c->fwd_ext = 1; c->fwd_block_n = pick_pair_block_n(T, s->d_out, 0, pairs); }
      }
    }
    c->stages = 6;
    c->dx_stages = 6;
    const long long fwd_t = static_cast<long long>(ceil_div(T, kPairBlockM)) * ceil_div(s->d_out, c->fwd_block_n);
    const long long dx_t = static_cast<long long>(ceil_div(T, kPairBlockM)) * ceil_div(s->d_in, c->dx_block_n);
    const long long fwd_items = fwd_t * c->split_k, dx_items = dx_t * c->dx_split_k;
    c->fwd_ctas = 2 * static_cast<int>(fwd_items < pairs ? fwd_items : pairs);
    c->dx_ctas = 2 * static_cast<int>(dx_items < pairs ? dx_items : pairs);
  } else {
    const long long fwd_tiles = static_cast<long long>(ceil_div(T, kBlockM)) * ceil_div(s->d_out, c->fwd_block_n);
    const long long dx_tiles = static_cast<long long>(ceil_div(T, kBlockM)) * ceil_div(s->d_in, c->dx_block_n);
    c->fwd_ctas = static_cast<int>(fwd_tiles < num_sms ? fwd_tiles : num_sms);
    c->dx_ctas = static_cast<int>(dx_tiles < num_sms ? dx_tiles : num_sms);
  }
  if (num_sms >= 2) {
    // dense weight gradient dW = dY^T X (always on CTA pairs): output rows = d_out, columns = d_in, contraction over
    // the tokens; same tile-width and split rules as the GEMMs above
    const int pairs = num_sms / 2;
    c->dw_block_n = pick_pair_block_n(s->d_out, s->d_in, 0, pairs);
    const long long tiles = static_cast<long long>(ceil_div(s->d_out, kPairBlockM)) * ceil_div(s->d_in, c->dw_block_n);
    const int kb = ceil_div(T, kBlockK);
    long long sp = 1;
    if (tiles * 4 <= pairs && kb >= 64) {
      sp = pairs / tiles;
      if (sp > kb / 16) sp = kb / 16;
      if (sp > 8) sp = 8;
      if (sp < 1) sp = 1;
    }
    c->dw_split_k = static_cast<int>(sp);
    const long long items = tiles * sp;
    c->dw_ctas = 2 * static_cast<int>(items < pairs ? items : pairs);
  } else {
    c->dw_block_n = 0;
    c->dw_split_k = 1;
    c->dw_ctas = 0;
  }
  if (const char* f = std::getenv("LORA_FORCE_STAGES")) {   // tuning knob: shallower rings
    const int v = std::atoi(f);
    if (v >= 2 && v <= c->stages) c->stages = v;
    if (v >= 2 && v <= c->dx_stages) c->dx_stages = v;
  }
  if (const char* f = std::getenv("LORA_FORCE_CTAS")) {   // tuning knob: cap the persistent GEMM grids
    const int v = std::atoi(f) / c->cta_group * c->cta_group;
    if (v >= c->cta_group) {
      if (v < c->fwd_ctas) c->fwd_ctas = v;
      if (v < c->dx_ctas) c->dx_ctas = v;
    }
  }
  const GradGrid ga = pick_grad_grid(T, s->d_in, c->r_pad, true, num_sms);
  const GradGrid gb = pick_grad_grid(T, s->d_out, c->r_pad, false, num_sms);
  c->grad_feat_chunk = ga.feat_chunk;
  c->grad_stages = ga.stages;
  c->db_stages = gb.stages;
  c->da_feat_chunks = ga.n_feat;
  c->da_token_chunks = ga.n_tok;
  c->db_feat_chunks = gb.n_feat;
  c->db_token_chunks = gb.n_tok;
  c->db_feat_chunk = gb.feat_chunk;
  // Overlapped backward (lora_linear_bwd), opt-in through LORA_OVERLAP_SMS = R: the tensor-bound dX GEMM leaves R SMs free
  // and the two HBM-bound adapter-gradient passes run on them at the same time on a second stream.  Measured (ms per
  // step, serial vs overlapped, same run): 8192 x 4096 x 4096 0.442 / 0.426 (R = 16), 0.437 (R = 24), 0.530 (R = 8: the
  // passes reach only ~40 GB/s per SM and outlast the GEMM); 16384 x 4096 x 14336 2.909 / 2.907; 16384 x 14336 x 4096
  // r = 64 3.055 / 3.159.  A gain within the run-to-run spread on the short step and none or a loss under the power cap
  // of the long ones, so the default stays the serial order.
  c->overlap_sms = 0;
  c->ov_dx_ctas = c->dx_ctas;
  c->ov_da_token_chunks = c->da_token_chunks;
  c->ov_db_token_chunks = c->db_token_chunks;
  if (c->cta_group == 2 && c->dx_split_k == 1) {
    const int pairs = num_sms / 2;
    int R = 0;
    if (const char* f = std::getenv("LORA_OVERLAP_SMS")) R = std::atoi(f) / 2 * 2;
    if (R >= 2 && R / 2 < pairs) {
      const long long dx_t = static_cast<long long>(ceil_div(T, kPairBlockM)) * ceil_div(s->d_in, c->dx_block_n);
      if (dx_t >= pairs) {
        c->overlap_sms = R;
        c->ov_dx_ctas = 2 * (pairs - R / 2);
        const int n_slabs = ceil_div(T, kGradSlab);
        auto tok = [&](int n_feat) {
          int n = R / n_feat;
          if (n < 1) n = 1;
          if (n > n_slabs) n = n_slabs;
          return n;
        };
        c->ov_da_token_chunks = tok(c->da_feat_chunks);
        c->ov_db_token_chunks = tok(c->db_feat_chunks);
        if (c->ov_da_token_chunks > c->da_token_chunks) c->ov_da_token_chunks = c->da_token_chunks;   // partials fit the workspace
        if (c->ov_db_token_chunks > c->db_token_chunks) c->ov_db_token_chunks = c->db_token_chunks;
      }
    }
  }
  {  // Q = dY B pre-pass of the CTA-pair backward
    const SideGrid q = pick_side_grid(T, s->d_out, num_sms);
    c->q_feat_chunk = q.feat_chunk;
    c->q_feat_chunks = q.n_feat;
    c->q_token_chunks = q.n_tok;
    c->q_stages = 4;
  }
  return LORA_OK;
}

// ------------------------------------------------------------------------------------------------
// backward workspace layout
// ------------------------------------------------------------------------------------------------
struct WsLayout {
  size_t qt, pt, q_part, p_part, da_part, db_part, split_part, total;
  int ld_t, c_pad_a, c_pad_b, n_slabs;
};

WsLayout ws_layout(const lora_shape_t& s, const lora_kernel_config_t& c) {
  WsLayout w;
  const long long T = s.T > 0 ? s.T : 1;
  w.ld_t = static_cast<int>(align_up(static_cast<size_t>(T), 64));
  w.c_pad_a = static_cast<int>(align_up(static_cast<size_t>(s.d_in), 32));
  w.c_pad_b = static_cast<int>(align_up(static_cast<size_t>(s.d_out), 32));
  w.n_slabs = ceil_div(T, kGradSlab);
  size_t off = 0;
  w.qt = off;       off += align_up(static_cast<size_t>(c.r_pad) * w.ld_t * 2, kAlign);
  w.pt = off;       off += align_up(static_cast<size_t>(c.r_pad) * w.ld_t * 2, kAlign);
  {
    int side_chunks = c.q_feat_chunks > c.db_feat_chunks ? c.q_feat_chunks : c.db_feat_chunks;
    if (side_chunks < 4) side_chunks = 4;   // the X A^T pre-pass of a K-extended forward uses at most 4 feature chunks
    w.q_part = off;
    off += align_up(static_cast<size_t>(side_chunks) * c.r_pad * w.ld_t * 4, kAlign);
  }
  w.p_part = off;   off += align_up(static_cast<size_t>(c.da_feat_chunks) * c.r_pad * w.ld_t * 4, kAlign);
  w.da_part = off;  off += align_up(static_cast<size_t>(c.da_token_chunks) * c.r_pad * w.c_pad_a * 4, kAlign);
  w.db_part = off;  off += align_up(static_cast<size_t>(c.db_token_chunks) * c.r_pad * w.c_pad_b * 4, kAlign);
  {
    const size_t f = c.split_k > 1 ? static_cast<size_t>(c.split_k) * T * s.d_out * 4 : 0;
    const size_t b = c.dx_split_k > 1 ? static_cast<size_t>(c.dx_split_k) * T * s.d_in * 4 : 0;
    const size_t g = c.dw_split_k > 1 ? static_cast<size_t>(c.dw_split_k) * s.d_out * s.d_in * 4 : 0;
    w.split_part = off;
    off += align_up(f > b ? (f > g ? f : g) : (b > g ? b : g), kAlign);
  }
  w.total = off;
  return w;
}

// ------------------------------------------------------------------------------------------------
// tensor maps
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess) return nullptr;
    if (q != cudaDriverEntryPointSuccess) return nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

// 2-D row-major tensor of `elem_bytes`-wide elements, 128-byte swizzle, zero fill outside the tensor.
// A tensor map is a pure function of (address, shape, pitch, box, type, swizzle), so encoded maps are kept in a small
// per-thread table: a step of the layer re-encodes the same ~40 maps every time, and on launch-bound shapes (a few
// hundred tokens) the driver's encode calls were the larger part of the host time per launch.
struct TmapKey {
  const void* ptr;
  uint64_t inner, outer, pitch;
  uint32_t box_inner, box_outer, dt, swz;
  bool operator==(const TmapKey& o) const {
    return ptr == o.ptr && inner == o.inner && outer == o.outer && pitch == o.pitch && box_inner == o.box_inner &&
           box_outer == o.box_outer && dt == o.dt && swz == o.swz;
  }
};
struct TmapSlot {
  bool used = false;
  TmapKey key;
  CUtensorMap map;
};
constexpr int kTmapCacheSlots = 512;        // direct-mapped; a colliding entry is simply re-encoded

bool make_tmap(CUtensorMap* m, const void* ptr, CUtensorMapDataType dt, int elem_bytes, uint64_t inner, uint64_t outer,
               uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_outer, bool swizzle128 = true) {
  static thread_local TmapSlot cache[kTmapCacheSlots];
  const TmapKey key{ptr, inner, outer, pitch_bytes, box_inner, box_outer, static_cast<uint32_t>(dt), swizzle128 ? 1u : 0u};
  uint64_t h = reinterpret_cast<uintptr_t>(ptr) * 0x9E3779B97F4A7C15ull;
  h ^= (inner * 0xC2B2AE3D27D4EB4Full) ^ (outer * 0x165667B19E3779F9ull) ^ (static_cast<uint64_t>(box_inner) << 40) ^
       (static_cast<uint64_t>(box_outer) << 20) ^ (pitch_bytes << 7) ^ key.dt ^ (key.swz << 5);
  TmapSlot& slot = cache[(h >> 32) % kTmapCacheSlots];
  if (slot.used && slot.key == key) {
    *m = slot.map;
    return true;
  }
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {inner, outer};
  const cuuint64_t strides[1] = {pitch_bytes};
  const cuuint32_t box[2] = {box_inner, box_outer};
  const cuuint32_t estr[2] = {1, 1};
  (void)elem_bytes;
  const CUresult r = fn(m, dt, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  slot.used = true;
  slot.key = key;
  slot.map = *m;
  return true;
}

bool make_bf16_tmap(CUtensorMap* m, const void* ptr, uint64_t inner, uint64_t outer, uint64_t pitch_elems,
                    uint32_t box_inner, uint32_t box_outer, bool swizzle128 = true) {
  return make_tmap(m, ptr, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, inner, outer, pitch_elems * 2, box_inner, box_outer,
                   swizzle128);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

// ------------------------------------------------------------------------------------------------
// plan
// ------------------------------------------------------------------------------------------------
struct lora_plan {
  lora_shape_t shape;
  lora_kernel_config_t cfg;
  WsLayout ws;
  int device;
  int num_sms;
  unsigned* d_status;   // 64 words of device memory
  void* workspace;
  size_t workspace_bytes;
  bool q_ready;          // set while lora_linear_bwd_saved_p runs: Qt was already produced by its dB kernel
  bool accumulate;       // dA / dB are added to instead of overwritten (lora_plan_set_grad_accumulation)
  bool q_staged;         // lora_linear_bwd_q ran: the next lora_linear_bwd_dx skips its own pre-pass
  cudaStream_t side_stream;   // overlapped backward: the adapter-gradient passes run here beside the dX GEMM
  cudaEvent_t ev_fork, ev_join;
  bool p_saved;          // the workspace holds Pt = s (X A^T)^T of the last forward call
  float p_saved_scale;
  long long wait_limit;  // SM clock ticks after which a device-side spin gives up (lora_plan_set_wait_limit)
};

namespace {

struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = (cudaSetDevice(dev) == cudaSuccess);
  }
  ~DeviceGuard() {
    if (switched) cudaSetDevice(prev);
  }
};

struct WsPtrs {
  uint8_t* base;
  __nv_bfloat16 *qt, *pt;
};

WsPtrs ws_ptrs(lora_plan* pl) {
  WsPtrs q;
  q.base = static_cast<uint8_t*>(pl->workspace);
  q.qt = reinterpret_cast<__nv_bfloat16*>(q.base + pl->ws.qt);
  q.pt = reinterpret_cast<__nv_bfloat16*>(q.base + pl->ws.pt);
  return q;
}

// Skinny side-product pass: out_t = s (S side^T)^T as bf16 [r_pad, ld_t], S = X with side = A [r, C] (K-major) or
// S = dY with side = B [C, r] (MN-major).  Streams S once; partials over feature chunks are summed in fixed order.
int launch_side_prepass(lora_plan* pl, const void* S, long long C, const void* side, bool side_mn, float scale,
                        __nv_bfloat16* out_t, cudaStream_t st) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  const WsLayout& w = pl->ws;
  CUtensorMap tmS, tmSide;
  bool ok = make_bf16_tmap(&tmS, S, C, s.T, C, 64, kGradSlab);
  if (side_mn) ok = ok && make_bf16_tmap(&tmSide, side, s.r, C, s.r, 64, 64);
  else ok = ok && make_bf16_tmap(&tmSide, side, C, s.r, C, 64, c.r_pad);
  if (!ok) return LORA_ERR_CUDA;
  const SideGrid sg = pick_side_grid(s.T, C, pl->num_sms);
  const int n_slabs = w.n_slabs;
  const int fc = sg.feat_chunk, nf = sg.n_feat, nt = sg.n_tok;
  GradParams g{};
  g.T = static_cast<int>(s.T);
  g.C = static_cast<int>(C);
  g.r = static_cast<int>(s.r);
  g.r_pad = c.r_pad;
  g.feat_chunk = fc;
  g.n_feat_chunks = nf;
  g.n_token_chunks = nt;
  g.n_slabs = n_slabs;
  g.stages = side_mn ? 4 : ((232448 - 4 * c.r_pad * 128 - 2048) / (kGradStageBytes + 2 * c.r_pad * 128) > 6
                                ? 6 : (232448 - 4 * c.r_pad * 128 - 2048) / (kGradStageBytes + 2 * c.r_pad * 128));
  g.with_p = 1;
  g.side_mn = side_mn ? 1 : 0;
  g.do_out = 0;
  g.scale = scale;
  g.p_part = reinterpret_cast<float*>(static_cast<uint8_t*>(pl->workspace) + w.q_part);
  g.pt_out = out_t;
  g.ld_t = w.ld_t;
  g.status = pl->d_status;
    g.wait_limit = pl->wait_limit;
  if (launch_grad(tmS, tmS, tmSide, g, st) != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(grad_is_direct(g) ? 1 : 2);
  return LORA_OK;
}

int launch_fwd(lora_plan* pl, const void* X, const void* W, const void* A, const void* B, float scale, void* Y,
               cudaStream_t st) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  const bool pair = c.cta_group == 2;
  const bool ext = pair && c.fwd_ext != 0;
  const bool have_ws = pl->workspace != nullptr && pl->workspace_bytes >= pl->ws.total;
  if (ext && !have_ws) return LORA_ERR_WORKSPACE;
  __nv_bfloat16* pt = have_ws ? ws_ptrs(pl).pt : nullptr;
  if (ext) {
    const int rc = launch_side_prepass(pl, X, s.d_in, A, false, scale, pt, st);   // Pt = s (X A^T)^T
    if (rc != LORA_OK) return rc;
  }
  const int half = (c.fwd_block_n + c.r_pad) / 2;
  CUtensorMap tmX, tmW, tmW1, tmA, tmB, tmY;
  bool ok = make_bf16_tmap(&tmX, X, s.d_in, s.T, s.d_in, 64, kBlockM);
  ok = ok && make_bf16_tmap(&tmW, W, s.d_in, s.d_out, s.d_in, 64, ext ? c.fwd_block_n / 2 : pair ? half : c.fwd_block_n);
  if (pair && !ext) ok = ok && make_bf16_tmap(&tmW1, W, s.d_in, s.d_out, s.d_in, 64, c.fwd_block_n - half);
  if (ext) ok = ok && make_bf16_tmap(&tmA, pt, s.T, c.r_pad, pl->ws.ld_t, 64, c.r_pad);
  else ok = ok && make_bf16_tmap(&tmA, A, s.d_in, s.r, s.d_in, 64, c.r_pad);
  ok = ok && make_bf16_tmap(&tmB, B, s.r, s.d_out, s.r, 64, pair ? c.fwd_block_n / 2 : c.fwd_block_n);
  ok = ok && make_bf16_tmap(&tmY, Y, s.d_out, s.T, s.d_out, 64, kBlockM);
  if (!ok) return LORA_ERR_CUDA;
  GemmParams p{};
  p.out = static_cast<__nv_bfloat16*>(Y);
  p.ld_out = static_cast<int>(s.d_out);
  p.M = static_cast<int>(s.T);
  p.N = static_cast<int>(s.d_out);
  p.K = static_cast<int>(s.d_in);
  p.r_pad = c.r_pad;
  p.block_n = c.fwd_block_n;
  p.tiles_m = ceil_div(s.T, c.block_m);
  p.tiles_n = ceil_div(s.d_out, c.fwd_block_n);
  p.num_tiles = p.tiles_m * p.tiles_n;
  p.kblocks = ceil_div(s.d_in, kBlockK);
  p.group_m = c.group_m;
  p.stages = c.stages;
  p.tail_delay = c.tail_delay;
  p.prefetch_dist = c.prefetch_dist;
  p.scale = scale;
  // with a registered workspace the CTA-pair forward leaves Pt = s (X A^T)^T there for lora_linear_bwd_saved_p
  const int kb_total = ceil_div(s.d_in, kBlockK);
  p.kb_per_split = ext ? ceil_div(kb_total, c.split_k) : kb_total;
  p.split_k = ext ? ceil_div(kb_total, p.kb_per_split) : 1;
  p.part = (p.split_k > 1) ? reinterpret_cast<float*>(static_cast<uint8_t*>(pl->workspace) + pl->ws.split_part) : nullptr;
  p.rt_out = (pair && !ext) ? pt : nullptr;
  p.ld_rt = pl->ws.ld_t;
  p.status = pl->d_status;
    p.wait_limit = pl->wait_limit;
  const cudaError_t le = ext    ? launch_gemm_pair_fwd_ext(tmX, tmW, tmA, tmB, tmY, p, c.fwd_ctas, st)
                         : pair ? launch_gemm_pair_fwd(tmX, tmW, tmW1, tmA, tmB, tmY, p, c.fwd_ctas, st)
                                : launch_gemm_fwd(tmX, tmW, tmA, tmB, tmY, p, c.fwd_ctas, st);
  if (le != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  if (p.split_k > 1) {
    if (launch_splitk_reduce(p.part, static_cast<__nv_bfloat16*>(Y), static_cast<long long>(s.T) * s.d_out, p.split_k, st) !=
        cudaSuccess)
      return LORA_ERR_CUDA;
    g_launches.fetch_add(1);
  }
  pl->p_saved = pair && pt != nullptr;
  pl->p_saved_scale = scale;
  return LORA_OK;
}

// ---- dX = dY W + s (dY B) A ; also leaves Qt = s (dY B)^T in the workspace ----
int launch_dx(lora_plan* pl, const void* dY, const void* W, const void* A, const void* B, float scale, void* dX,
              cudaStream_t st, int ctas_override = 0) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  const WsLayout& w = pl->ws;
  const WsPtrs q = ws_ptrs(pl);
  __nv_bfloat16* qt = q.qt;
  if (c.cta_group == 2 && !pl->q_ready) {
    // ---- pre-pass: Qt = s (dY B)^T, dY streamed once by the skinny kernel (side product only) ----
    const int rc = launch_side_prepass(pl, dY, s.d_out, B, true, scale, qt, st);
    if (rc != LORA_OK) return rc;
  }
  {
    CUtensorMap tmdY, tmW, tmB, tmA, tmdX;
    bool ok = make_bf16_tmap(&tmdY, dY, s.d_out, s.T, s.d_out, 64, kBlockM);
    ok = ok && make_bf16_tmap(&tmW, W, s.d_in, s.d_out, s.d_in, 64, 64);
    const bool pair = c.cta_group == 2;
    if (pair) ok = ok && make_bf16_tmap(&tmB, qt, s.T, c.r_pad, w.ld_t, 64, c.r_pad);   // Qt from the pre-pass below
    else ok = ok && make_bf16_tmap(&tmB, B, s.r, s.d_out, s.r, 64, 64);
    ok = ok && make_bf16_tmap(&tmA, A, s.d_in, s.r, s.d_in, 64, c.r_pad);
    ok = ok && make_bf16_tmap(&tmdX, dX, s.d_in, s.T, s.d_in, 64, kBlockM);
    if (!ok) return LORA_ERR_CUDA;
    GemmParams p{};
    p.out = static_cast<__nv_bfloat16*>(dX);
    p.ld_out = static_cast<int>(s.d_in);
    p.M = static_cast<int>(s.T);
    p.N = static_cast<int>(s.d_in);
    p.K = static_cast<int>(s.d_out);
    p.r_pad = c.r_pad;
    p.block_n = c.dx_block_n;
    p.tiles_m = ceil_div(s.T, c.block_m);
    p.tiles_n = ceil_div(s.d_in, c.dx_block_n);
    p.num_tiles = p.tiles_m * p.tiles_n;
    p.kblocks = ceil_div(s.d_out, kBlockK);
    p.group_m = c.group_m;
    p.stages = c.dx_stages;
    p.tail_delay = c.tail_delay;
    p.prefetch_dist = c.prefetch_dist;
    p.scale = scale;
    const int kb_total = ceil_div(s.d_out, kBlockK);
    p.kb_per_split = pair ? ceil_div(kb_total, c.dx_split_k) : kb_total;
    p.split_k = pair ? ceil_div(kb_total, p.kb_per_split) : 1;
    p.part = (p.split_k > 1) ? reinterpret_cast<float*>(q.base + w.split_part) : nullptr;
    p.rt_out = pair ? nullptr : qt;     // the single-CTA kernel computes Q itself and hands it on
    p.ld_rt = w.ld_t;
    p.status = pl->d_status;
    p.wait_limit = pl->wait_limit;
    const int ctas = ctas_override > 0 ? ctas_override : c.dx_ctas;
    const cudaError_t le = pair ? launch_gemm_pair_dx(tmdY, tmW, tmB, tmA, tmdX, p, ctas, st)
                                : launch_gemm_dx(tmdY, tmW, tmB, tmA, tmdX, p, ctas, st);
    if (le != cudaSuccess) return LORA_ERR_CUDA;
    g_launches.fetch_add(1);
    if (p.split_k > 1) {
      if (launch_splitk_reduce(p.part, static_cast<__nv_bfloat16*>(dX), static_cast<long long>(s.T) * s.d_in, p.split_k, st) !=
          cudaSuccess)
        return LORA_ERR_CUDA;
      g_launches.fetch_add(1);
    }
  }
  return LORA_OK;
}

// ---- dA = Qt-contraction over X; recomputes X A^T and leaves Pt = s (X A^T)^T ----
int launch_da(lora_plan* pl, const void* X, const void* A, float scale, void* dA, cudaStream_t st, bool with_p = true,
              int tok_override = 0) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  const WsLayout& w = pl->ws;
  const WsPtrs q = ws_ptrs(pl);
  uint8_t* ws = q.base;
  __nv_bfloat16 *qt = q.qt, *pt = q.pt;
  {
    CUtensorMap tmS, tmR, tmA;
    bool ok = make_bf16_tmap(&tmS, X, s.d_in, s.T, s.d_in, 64, kGradSlab);
    ok = ok && make_bf16_tmap(&tmR, qt, s.T, c.r_pad, w.ld_t, 64, c.r_pad);
    ok = ok && make_bf16_tmap(&tmA, A, s.d_in, s.r, s.d_in, 64, c.r_pad);
    if (!ok) return LORA_ERR_CUDA;
    GradParams g{};
    g.T = static_cast<int>(s.T);
    g.C = static_cast<int>(s.d_in);
    g.r = static_cast<int>(s.r);
    g.r_pad = c.r_pad;
    g.feat_chunk = c.grad_feat_chunk;
    g.n_feat_chunks = c.da_feat_chunks;
    g.n_token_chunks = tok_override > 0 ? tok_override : c.da_token_chunks;
    g.n_slabs = w.n_slabs;
    g.stages = with_p ? c.grad_stages : c.db_stages;
    g.with_p = with_p ? 1 : 0;
    g.side_mn = 0;
    g.do_out = 1;
    g.out_is_da = 1;
    g.accumulate = pl->accumulate ? 1 : 0;
    g.scale = scale;
    g.out = static_cast<float*>(dA);
    g.out_part = reinterpret_cast<float*>(ws + w.da_part);
    g.c_pad = w.c_pad_a;
    g.p_part = reinterpret_cast<float*>(ws + w.p_part);
    g.pt_out = pt;
    g.ld_t = w.ld_t;
    g.status = pl->d_status;
    g.wait_limit = pl->wait_limit;
    if (launch_grad(tmS, tmR, tmA, g, st) != cudaSuccess) return LORA_ERR_CUDA;
    g_launches.fetch_add(grad_is_direct(g) ? 1 : 2);
  }
  return LORA_OK;
}

// ---- dB = Pt-contraction over dY ----
int launch_db(lora_plan* pl, const void* dY, float scale, void* dB, cudaStream_t st, const void* B_for_q = nullptr,
              int tok_override = 0) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  const WsLayout& w = pl->ws;
  const WsPtrs q = ws_ptrs(pl);
  uint8_t* ws = q.base;
  __nv_bfloat16* pt = q.pt;
  {
    const bool with_q = B_for_q != nullptr;     // also leave Qt = s (dY B)^T (saved-P backward)
    CUtensorMap tmS, tmR, tmSide;
    bool ok = make_bf16_tmap(&tmS, dY, s.d_out, s.T, s.d_out, 64, kGradSlab);
    ok = ok && make_bf16_tmap(&tmR, pt, s.T, c.r_pad, w.ld_t, 64, c.r_pad);
    if (with_q) ok = ok && make_bf16_tmap(&tmSide, B_for_q, s.r, s.d_out, s.r, 64, 64);
    if (!ok) return LORA_ERR_CUDA;
    GradParams g{};
    g.T = static_cast<int>(s.T);
    g.C = static_cast<int>(s.d_out);
    g.r = static_cast<int>(s.r);
    g.r_pad = c.r_pad;
    g.feat_chunk = c.db_feat_chunk;
    g.n_feat_chunks = c.db_feat_chunks;
    g.n_token_chunks = tok_override > 0 ? tok_override : c.db_token_chunks;
    g.n_slabs = w.n_slabs;
    g.stages = with_q ? 4 : c.db_stages;
    g.with_p = with_q ? 1 : 0;
    g.side_mn = with_q ? 1 : 0;
    g.do_out = 1;
    g.out_is_da = 0;
    g.accumulate = pl->accumulate ? 1 : 0;
    g.scale = scale;
    g.out = static_cast<float*>(dB);
    g.out_part = reinterpret_cast<float*>(ws + w.db_part);
    g.c_pad = w.c_pad_b;
    g.p_part = with_q ? reinterpret_cast<float*>(ws + w.q_part) : nullptr;
    g.pt_out = with_q ? q.qt : nullptr;
    g.ld_t = w.ld_t;
    g.status = pl->d_status;
    g.wait_limit = pl->wait_limit;
    if (launch_grad(tmS, tmR, with_q ? tmSide : tmR, g, st) != cudaSuccess) return LORA_ERR_CUDA;
    g_launches.fetch_add(grad_is_direct(g) ? 1 : 2);
  }
  return LORA_OK;
}

// ---- NF4 frozen weight (Q+LoRA): both GEMMs run K-extended on CTA pairs with the dequantising kernel variant ----
bool make_nf4_tmaps(CUtensorMap* tmCodes, CUtensorMap* tmAbsmax, const void* codes, const void* absmax, const lora_shape_t& s,
                    bool backward) {
  // codes [d_out, d_in / 2] uint8 (no swizzle): forward box = 32 bytes (one block) x 128 rows, backward 64 bytes x 64 rows;
  // absmax [d_in / 64, d_out] float: forward box = 128 rows' scales of one block, backward 64 rows' scales of two blocks
  bool ok = make_tmap(tmCodes, codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, s.d_in / 2, s.d_out, s.d_in / 2, backward ? 64 : 32,
                      backward ? 64 : 128, false);
  ok = ok && make_tmap(tmAbsmax, absmax, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, s.d_out, s.d_in / kNf4Block, s.d_out * 4,
                       backward ? 64 : 128, backward ? 2 : 1, false);
  return ok;
}

int launch_fwd_nf4(lora_plan* pl, const void* X, const void* codes, const void* absmax, const void* A, const void* B,
                   float scale, void* Y, cudaStream_t st) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  __nv_bfloat16* pt = ws_ptrs(pl).pt;
  int rc = launch_side_prepass(pl, X, s.d_in, A, false, scale, pt, st);   // Pt = s (X A^T)^T
  if (rc != LORA_OK) return rc;
  const int pairs = pl->num_sms / 2;
  const int bn = pick_pair_block_n(s.T, s.d_out, 0, pairs);
  CUtensorMap tmX, tmCodes, tmAbsmax, tmPt, tmB, tmY;
  bool ok = make_bf16_tmap(&tmX, X, s.d_in, s.T, s.d_in, 64, kBlockM);
  ok = ok && make_nf4_tmaps(&tmCodes, &tmAbsmax, codes, absmax, s, false);
  ok = ok && make_bf16_tmap(&tmPt, pt, s.T, c.r_pad, pl->ws.ld_t, 64, c.r_pad);
  ok = ok && make_bf16_tmap(&tmB, B, s.r, s.d_out, s.r, 64, bn / 2);
  ok = ok && make_bf16_tmap(&tmY, Y, s.d_out, s.T, s.d_out, 64, kBlockM);
  if (!ok) return LORA_ERR_CUDA;
  GemmParams p{};
  p.out = static_cast<__nv_bfloat16*>(Y);
  p.ld_out = static_cast<int>(s.d_out);
  p.M = static_cast<int>(s.T);
  p.N = static_cast<int>(s.d_out);
  p.K = static_cast<int>(s.d_in);
  p.r_pad = c.r_pad;
  p.block_n = bn;
  p.tiles_m = ceil_div(s.T, kPairBlockM);
  p.tiles_n = ceil_div(s.d_out, bn);
  p.num_tiles = p.tiles_m * p.tiles_n;
  p.kblocks = ceil_div(s.d_in, kBlockK);
  p.group_m = c.group_m;
  p.stages = 5;                       // one stage less than the bf16 kernels: the code ring and the level table need the room
  p.tail_delay = c.tail_delay;
  p.scale = scale;
  p.kb_per_split = p.kblocks;
  p.split_k = 1;
  p.status = pl->d_status;
    p.wait_limit = pl->wait_limit;
  const int ctas = 2 * (p.num_tiles < pairs ? p.num_tiles : pairs);
  if (launch_gemm_pair_fwd_nf4(tmX, tmCodes, tmAbsmax, tmPt, tmB, tmY, p, ctas, st) != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  pl->p_saved = false;
  return LORA_OK;
}

int launch_dx_nf4(lora_plan* pl, const void* dY, const void* codes, const void* absmax, const void* A, const void* B,
                  float scale, void* dX, cudaStream_t st) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  __nv_bfloat16* qt = ws_ptrs(pl).qt;
  int rc = launch_side_prepass(pl, dY, s.d_out, B, true, scale, qt, st);   // Qt = s (dY B)^T
  if (rc != LORA_OK) return rc;
  const int pairs = pl->num_sms / 2;
  const int bn = 256;                 // each CTA's 128 weight columns are two whole quantisation blocks
  CUtensorMap tmdY, tmCodes, tmAbsmax, tmQt, tmA, tmdX;
  bool ok = make_bf16_tmap(&tmdY, dY, s.d_out, s.T, s.d_out, 64, kBlockM);
  ok = ok && make_nf4_tmaps(&tmCodes, &tmAbsmax, codes, absmax, s, true);
  ok = ok && make_bf16_tmap(&tmQt, qt, s.T, c.r_pad, pl->ws.ld_t, 64, c.r_pad);
  ok = ok && make_bf16_tmap(&tmA, A, s.d_in, s.r, s.d_in, 64, c.r_pad);
  ok = ok && make_bf16_tmap(&tmdX, dX, s.d_in, s.T, s.d_in, 64, kBlockM);
  if (!ok) return LORA_ERR_CUDA;
  GemmParams p{};
  p.out = static_cast<__nv_bfloat16*>(dX);
  p.ld_out = static_cast<int>(s.d_in);
  p.M = static_cast<int>(s.T);
  p.N = static_cast<int>(s.d_in);
  p.K = static_cast<int>(s.d_out);
  p.r_pad = c.r_pad;
  p.block_n = bn;
  p.tiles_m = ceil_div(s.T, kPairBlockM);
  p.tiles_n = ceil_div(s.d_in, bn);
  p.num_tiles = p.tiles_m * p.tiles_n;
  p.kblocks = ceil_div(s.d_out, kBlockK);
  p.group_m = c.group_m;
  p.stages = 5;
  p.tail_delay = c.tail_delay;
  p.scale = scale;
  p.kb_per_split = p.kblocks;
  p.split_k = 1;
  p.status = pl->d_status;
    p.wait_limit = pl->wait_limit;
  const int ctas = 2 * (p.num_tiles < pairs ? p.num_tiles : pairs);
  if (launch_gemm_pair_dx_nf4(tmdY, tmCodes, tmAbsmax, tmQt, tmA, tmdX, p, ctas, st) != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  return LORA_OK;
}

int check_nf4(const lora_plan* pl) {
  if (pl->cfg.cta_group != 2) return LORA_ERR_UNSUPPORTED_SHAPE;          // batches of at most 128 tokens: not covered
  if (pl->shape.d_in % kNf4Block != 0) return LORA_ERR_UNSUPPORTED_SHAPE;
  if (pl->workspace == nullptr || pl->workspace_bytes < pl->ws.total) return LORA_ERR_WORKSPACE;
  return LORA_OK;
}

// ---- dW = dY^T X (full fine-tuning): plain GEMM with both operands MN-major, contraction over the tokens ----
int launch_dw(lora_plan* pl, const void* dY, const void* X, void* dW, cudaStream_t st) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  CUtensorMap tmdY, tmX, tmdW;
  bool ok = make_bf16_tmap(&tmdY, dY, s.d_out, s.T, s.d_out, 64, 64);
  ok = ok && make_bf16_tmap(&tmX, X, s.d_in, s.T, s.d_in, 64, 64);
  ok = ok && make_bf16_tmap(&tmdW, dW, s.d_in, s.d_out, s.d_in, 64, kBlockM);
  if (!ok) return LORA_ERR_CUDA;
  GemmParams p{};
  p.out = static_cast<__nv_bfloat16*>(dW);
  p.ld_out = static_cast<int>(s.d_in);
  p.M = static_cast<int>(s.d_out);
  p.N = static_cast<int>(s.d_in);
  p.K = static_cast<int>(s.T);
  p.r_pad = 0;
  p.block_n = c.dw_block_n;
  p.tiles_m = ceil_div(s.d_out, kPairBlockM);
  p.tiles_n = ceil_div(s.d_in, c.dw_block_n);
  p.num_tiles = p.tiles_m * p.tiles_n;
  p.kblocks = ceil_div(s.T, kBlockK);
  p.group_m = c.group_m;
  p.stages = 6;
  p.tail_delay = c.tail_delay;
  p.scale = 1.f;
  p.kb_per_split = ceil_div(p.kblocks, c.dw_split_k);
  p.split_k = ceil_div(p.kblocks, p.kb_per_split);
  p.part = (p.split_k > 1) ? reinterpret_cast<float*>(static_cast<uint8_t*>(pl->workspace) + pl->ws.split_part) : nullptr;
  p.status = pl->d_status;
    p.wait_limit = pl->wait_limit;
  if (launch_gemm_pair_dw(tmdY, tmX, tmdW, p, c.dw_ctas, st) != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  if (p.split_k > 1) {
    if (launch_splitk_reduce(p.part, static_cast<__nv_bfloat16*>(dW), static_cast<long long>(s.d_out) * s.d_in, p.split_k, st) !=
        cudaSuccess)
      return LORA_ERR_CUDA;
    g_launches.fetch_add(1);
  }
  return LORA_OK;
}

}  // namespace

extern "C" {

int lora_select_config(const lora_shape_t* shape, int num_sms, lora_kernel_config_t* out) {
  return select_config(shape, num_sms, out);
}

int lora_workspace_bytes(const lora_shape_t* shape, int num_sms, size_t* bwd_bytes) {
  if (bwd_bytes == nullptr) return LORA_ERR_INVALID_ARG;
  lora_kernel_config_t c;
  const int rc = select_config(shape, num_sms, &c);
  if (rc != LORA_OK) return rc;
  *bwd_bytes = ws_layout(*shape, c).total;
  return LORA_OK;
}

int lora_plan_create(const lora_shape_t* shape, int device, lora_plan_t** out) {
  if (out == nullptr) return LORA_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = check_shape(shape);
  if (rc != LORA_OK) return rc;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || count <= 0) {
    cudaGetLastError();
    return LORA_ERR_NO_DEVICE;
  }
  if (device < 0 || device >= count) return LORA_ERR_INVALID_ARG;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return LORA_ERR_CUDA;
  if (prop.major != 10) return LORA_ERR_NO_DEVICE;
  DeviceGuard guard(device);
  lora_plan* pl = new (std::nothrow) lora_plan();
  if (pl == nullptr) return LORA_ERR_INVALID_ARG;
  pl->shape = *shape;
  pl->device = device;
  pl->num_sms = prop.multiProcessorCount;
  rc = select_config(shape, pl->num_sms, &pl->cfg);
  if (rc != LORA_OK) {
    delete pl;
    return rc;
  }
  pl->ws = ws_layout(*shape, pl->cfg);
  pl->workspace = nullptr;
  pl->workspace_bytes = 0;
  pl->q_ready = false;
  pl->q_staged = false;
  pl->accumulate = false;
  pl->p_saved = false;
  pl->p_saved_scale = 0.f;
  pl->wait_limit = kWaitLimitCycles;
  if (const char* f = std::getenv("LORA_DEBUG_WAIT_CAP")) {     // debugging: shorter limit, in SM clock ticks
    const long long v = std::atoll(f);
    if (v >= 1000) pl->wait_limit = v;
  }
  pl->d_status = nullptr;
  pl->side_stream = nullptr;
  pl->ev_fork = pl->ev_join = nullptr;
  if (pl->cfg.overlap_sms > 0 &&
      (cudaStreamCreateWithFlags(&pl->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
       cudaEventCreateWithFlags(&pl->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
       cudaEventCreateWithFlags(&pl->ev_join, cudaEventDisableTiming) != cudaSuccess)) {
    cudaGetLastError();
    pl->cfg.overlap_sms = 0;         // no second stream: fall back to the serial order
  }
  if (gemm_configure() != cudaSuccess || gemm_pair_configure() != cudaSuccess || grad_configure() != cudaSuccess || encode_fn() == nullptr ||
      cudaMalloc(&pl->d_status, 256) != cudaSuccess || cudaMemset(pl->d_status, 0, 256) != cudaSuccess) {
    cudaGetLastError();
    if (pl->d_status) cudaFree(pl->d_status);
    delete pl;
    return LORA_ERR_CUDA;
  }
  *out = pl;
  return LORA_OK;
}

int lora_plan_destroy(lora_plan_t* plan) {
  if (plan == nullptr) return LORA_ERR_INVALID_ARG;
  DeviceGuard guard(plan->device);
  if (plan->d_status) cudaFree(plan->d_status);
  if (plan->ev_fork) cudaEventDestroy(plan->ev_fork);
  if (plan->ev_join) cudaEventDestroy(plan->ev_join);
  if (plan->side_stream) cudaStreamDestroy(plan->side_stream);
  delete plan;
  return LORA_OK;
}

int lora_plan_workspace_bytes(const lora_plan_t* plan, size_t* fwd_bytes, size_t* bwd_bytes) {
  if (plan == nullptr) return LORA_ERR_INVALID_ARG;
  if (fwd_bytes) *fwd_bytes = (plan->cfg.cta_group == 2 && plan->cfg.fwd_ext) ? plan->ws.total : 0;
  if (bwd_bytes) *bwd_bytes = plan->ws.total;
  return LORA_OK;
}

int lora_plan_set_workspace(lora_plan_t* plan, void* dev_ptr, size_t bytes) {
  if (plan == nullptr) return LORA_ERR_INVALID_ARG;
  if (dev_ptr == nullptr) {
    plan->workspace = nullptr;
    plan->workspace_bytes = 0;
    return bytes == 0 ? LORA_OK : LORA_ERR_INVALID_ARG;
  }
  if ((reinterpret_cast<uintptr_t>(dev_ptr) & (kAlign - 1)) != 0) return LORA_ERR_MISALIGNED;
  if (bytes < plan->ws.total) return LORA_ERR_WORKSPACE;
  plan->workspace = dev_ptr;
  plan->workspace_bytes = bytes;
  plan->p_saved = false;
  plan->q_staged = false;
  return LORA_OK;
}

int lora_plan_set_grad_accumulation(lora_plan_t* plan, int enable) {
  if (plan == nullptr) return LORA_ERR_INVALID_ARG;
  plan->accumulate = enable != 0;
  return LORA_OK;
}

int lora_plan_set_wait_limit(lora_plan_t* plan, int64_t cycles) {
  if (plan == nullptr || cycles < 0) return LORA_ERR_INVALID_ARG;
  plan->wait_limit = cycles == 0 ? kWaitLimitCycles : (cycles < 1000 ? 1000 : cycles);
  return LORA_OK;
}

int lora_debug_starved_wait(lora_plan_t* plan, const void* S, int64_t T, int64_t C, void* out, void* stream) {
  if (plan == nullptr || S == nullptr || out == nullptr) return LORA_ERR_INVALID_ARG;
  if (T < 1 || T > 1024 || C < 8 || C > 512 || C % 8 != 0) return LORA_ERR_UNSUPPORTED_SHAPE;
  if (!aligned16(S) || !aligned16(out)) return LORA_ERR_MISALIGNED;
  DeviceGuard guard(plan->device);
  const int r_pad = plan->cfg.r_pad;
  CUtensorMap tmS;
  if (!make_bf16_tmap(&tmS, S, C, T, C, 64, kGradSlab)) return LORA_ERR_CUDA;
  GradParams g{};
  g.T = static_cast<int>(T);
  g.C = static_cast<int>(C);
  g.r = static_cast<int>(plan->shape.r);
  g.r_pad = r_pad;
  g.feat_chunk = ceil_div(C, 128) * 128;
  g.n_feat_chunks = 1;
  g.n_token_chunks = 1;              // one CTA, direct mode: nothing but `status` can be written
  g.n_slabs = ceil_div(T, kGradSlab);
  g.stages = 2;
  g.do_out = 1;
  g.scale = 1.f;
  g.out = static_cast<float*>(out);
  g.c_pad = static_cast<int>(C);
  g.ld_t = static_cast<int>(T);
  g.status = plan->d_status;
  g.wait_limit = plan->wait_limit;
  g.debug_no_second_factor = 1;      // the MMA warp never receives its second factor: its bounded wait runs out
  if (launch_grad(tmS, tmS, tmS, g, static_cast<cudaStream_t>(stream)) != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  return LORA_OK;
}

int lora_plan_get_config(const lora_plan_t* plan, lora_kernel_config_t* out) {
  if (plan == nullptr || out == nullptr) return LORA_ERR_INVALID_ARG;
  *out = plan->cfg;
  return LORA_OK;
}

int lora_plan_describe(const lora_plan_t* plan, char* buf, size_t n) {
  if (plan == nullptr || buf == nullptr || n == 0) return LORA_ERR_INVALID_ARG;
  const lora_kernel_config_t& c = plan->cfg;
  std::snprintf(buf, n,
                "T=%lld d_in=%lld d_out=%lld r=%lld | sms=%d cta_group=%d tile fwd %dx%dx64 dx %dx%dx64 stages=%d/%d group_m=%d "
                "split_k=%d/%d r_pad=%d ctas fwd=%d dx=%d tail_delay=%d | grad chunk=%d/%d stages=%d/%d dA grid=%dx%d dB grid=%dx%d "
                "| bwd workspace=%zu B",
                (long long)plan->shape.T, (long long)plan->shape.d_in, (long long)plan->shape.d_out,
                (long long)plan->shape.r, plan->num_sms, c.cta_group, c.block_m, c.fwd_block_n, c.block_m, c.dx_block_n,
                c.stages, c.dx_stages, c.group_m, c.split_k, c.dx_split_k,
                c.r_pad, c.fwd_ctas, c.dx_ctas, c.tail_delay, c.grad_feat_chunk, c.db_feat_chunk, c.grad_stages, c.db_stages,
                c.da_feat_chunks,
                c.da_token_chunks, c.db_feat_chunks, c.db_token_chunks, plan->ws.total);
  return LORA_OK;
}

int lora_linear_fwd(lora_plan_t* plan, const void* X, const void* W, const void* A, const void* B, float scale,
                    void* Y, void* stream) {
  if (plan == nullptr) return LORA_ERR_INVALID_ARG;
  if (plan->shape.T == 0) return LORA_OK;
  if (!X || !W || !A || !B || !Y) return LORA_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(W) || !aligned16(A) || !aligned16(B) || !aligned16(Y)) return LORA_ERR_MISALIGNED;
  DeviceGuard guard(plan->device);
  return launch_fwd(plan, X, W, A, B, scale, Y, static_cast<cudaStream_t>(stream));
}

int lora_linear_bwd(lora_plan_t* plan, const void* dY, const void* X, const void* W, const void* A, const void* B,
                    float scale, void* dX, void* dA, void* dB, void* stream) {
  if (plan == nullptr) return LORA_ERR_INVALID_ARG;
  if (!dA || !dB) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dA) || !aligned16(dB)) return LORA_ERR_MISALIGNED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  DeviceGuard guard(plan->device);
  if (plan->shape.T == 0) {   // empty batch: the sums over tokens are empty
    if (plan->accumulate) return LORA_OK;
    if (cudaMemsetAsync(dA, 0, sizeof(float) * plan->shape.r * plan->shape.d_in, st) != cudaSuccess ||
        cudaMemsetAsync(dB, 0, sizeof(float) * plan->shape.d_out * plan->shape.r, st) != cudaSuccess)
      return LORA_ERR_CUDA;
    return LORA_OK;
  }
  if (!dY || !X || !W || !A || !B || !dX) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(X) || !aligned16(W) || !aligned16(A) || !aligned16(B) || !aligned16(dX))
    return LORA_ERR_MISALIGNED;
  if (plan->workspace == nullptr || plan->workspace_bytes < plan->ws.total) return LORA_ERR_WORKSPACE;
  plan->q_staged = false;      // this call overwrites the staged s (dY B)^T
  if (plan->cfg.overlap_sms > 0) {
    // dY B pre-pass, then the dX GEMM on `stream` beside dA -> dB on the plan's second stream (fork / join by events)
    const lora_kernel_config_t& c = plan->cfg;
    int rc = launch_side_prepass(plan, dY, plan->shape.d_out, B, true, scale, ws_ptrs(plan).qt, st);
    if (rc != LORA_OK) return rc;
    if (cudaEventRecord(plan->ev_fork, st) != cudaSuccess || cudaStreamWaitEvent(plan->side_stream, plan->ev_fork, 0) != cudaSuccess)
      return LORA_ERR_CUDA;
    plan->q_ready = true;
    rc = launch_dx(plan, dY, W, A, B, scale, dX, st, c.ov_dx_ctas);
    plan->q_ready = false;
    if (rc == LORA_OK) rc = launch_da(plan, X, A, scale, dA, plan->side_stream, true, c.ov_da_token_chunks);
    if (rc == LORA_OK) rc = launch_db(plan, dY, scale, dB, plan->side_stream, nullptr, c.ov_db_token_chunks);
    // join even after a failed launch, so that `stream` never runs ahead of work already queued on the second stream
    if (cudaEventRecord(plan->ev_join, plan->side_stream) != cudaSuccess || cudaStreamWaitEvent(st, plan->ev_join, 0) != cudaSuccess)
      return LORA_ERR_CUDA;
    return rc;
  }
  int rc = launch_dx(plan, dY, W, A, B, scale, dX, st);
  if (rc == LORA_OK) rc = launch_da(plan, X, A, scale, dA, st);
  if (rc == LORA_OK) rc = launch_db(plan, dY, scale, dB, st);
  return rc;
}

int lora_linear_bwd_saved_p(lora_plan_t* plan, const void* dY, const void* X, const void* W, const void* A, const void* B,
                            float scale, void* dX, void* dA, void* dB, void* stream) {
  if (plan == nullptr) return LORA_ERR_INVALID_ARG;
  if (plan->shape.T == 0 || plan->cfg.cta_group != 2)      // nothing was saved for these: same as the plain call
    return lora_linear_bwd(plan, dY, X, W, A, B, scale, dX, dA, dB, stream);
  if (!dY || !X || !W || !A || !B || !dX || !dA || !dB) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(X) || !aligned16(W) || !aligned16(A) || !aligned16(B) || !aligned16(dX) ||
      !aligned16(dA) || !aligned16(dB))
    return LORA_ERR_MISALIGNED;
  if (plan->workspace == nullptr || plan->workspace_bytes < plan->ws.total) return LORA_ERR_WORKSPACE;
  if (!plan->p_saved || plan->p_saved_scale != scale) return LORA_ERR_INVALID_ARG;   // no forward result to reuse
  plan->q_staged = false;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  DeviceGuard guard(plan->device);
  int rc = launch_db(plan, dY, scale, dB, st, B);          // dB from the saved Pt; leaves Qt
  if (rc == LORA_OK) {
    plan->q_ready = true;
    rc = launch_dx(plan, dY, W, A, B, scale, dX, st);      // K-extended GEMM only
    plan->q_ready = false;
  }
  if (rc == LORA_OK) rc = launch_da(plan, X, A, scale, dA, st, false);
  return rc;
}

int lora_linear_bwd_q(lora_plan_t* plan, const void* dY, const void* B, float scale, void* stream) {
  if (plan == nullptr) return LORA_ERR_INVALID_ARG;
  if (plan->shape.T == 0 || plan->cfg.cta_group != 2) return LORA_OK;   // small batches: the dX kernel computes dY B itself
  if (!dY || !B) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(B)) return LORA_ERR_MISALIGNED;
  if (plan->workspace == nullptr || plan->workspace_bytes < plan->ws.total) return LORA_ERR_WORKSPACE;
  DeviceGuard guard(plan->device);
  const int rc = launch_side_prepass(plan, dY, plan->shape.d_out, B, true, scale, ws_ptrs(plan).qt, static_cast<cudaStream_t>(stream));
  if (rc == LORA_OK) plan->q_staged = true;
  return rc;
}

int lora_linear_bwd_dx(lora_plan_t* plan, const void* dY, const void* W, const void* A, const void* B, float scale,
                       void* dX, void* stream) {
  if (plan == nullptr) return LORA_ERR_INVALID_ARG;
  if (plan->shape.T == 0) return LORA_OK;
  if (!dY || !W || !A || !B || !dX) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(W) || !aligned16(A) || !aligned16(B) || !aligned16(dX)) return LORA_ERR_MISALIGNED;
  if (plan->workspace == nullptr || plan->workspace_bytes < plan->ws.total) return LORA_ERR_WORKSPACE;
  DeviceGuard guard(plan->device);
  plan->q_ready = plan->q_staged;          // lora_linear_bwd_q already left s (dY B)^T in the workspace
  plan->q_staged = false;
  const int rc = launch_dx(plan, dY, W, A, B, scale, dX, static_cast<cudaStream_t>(stream));
  plan->q_ready = false;
  return rc;
}

int lora_linear_bwd_da(lora_plan_t* plan, const void* X, const void* A, float scale, void* dA, void* stream) {
  if (plan == nullptr || !dA) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dA)) return LORA_ERR_MISALIGNED;
  DeviceGuard guard(plan->device);
  if (plan->shape.T == 0 && plan->accumulate) return LORA_OK;
  if (plan->shape.T == 0)
    return cudaMemsetAsync(dA, 0, sizeof(float) * plan->shape.r * plan->shape.d_in, static_cast<cudaStream_t>(stream)) ==
                   cudaSuccess ? LORA_OK : LORA_ERR_CUDA;
  if (!X || !A) return LORA_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(A)) return LORA_ERR_MISALIGNED;
  if (plan->workspace == nullptr || plan->workspace_bytes < plan->ws.total) return LORA_ERR_WORKSPACE;
  return launch_da(plan, X, A, scale, dA, static_cast<cudaStream_t>(stream));
}

int lora_linear_bwd_db(lora_plan_t* plan, const void* dY, float scale, void* dB, void* stream) {
  if (plan == nullptr || !dB) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dB)) return LORA_ERR_MISALIGNED;
  DeviceGuard guard(plan->device);
  if (plan->shape.T == 0 && plan->accumulate) return LORA_OK;
  if (plan->shape.T == 0)
    return cudaMemsetAsync(dB, 0, sizeof(float) * plan->shape.d_out * plan->shape.r, static_cast<cudaStream_t>(stream)) ==
                   cudaSuccess ? LORA_OK : LORA_ERR_CUDA;
  if (!dY) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dY)) return LORA_ERR_MISALIGNED;
  if (plan->workspace == nullptr || plan->workspace_bytes < plan->ws.total) return LORA_ERR_WORKSPACE;
  return launch_db(plan, dY, scale, dB, static_cast<cudaStream_t>(stream));
}

int lora_nf4_quantize(const void* W, int64_t d_out, int64_t d_in, void* codes, void* absmax, void* stream) {
  if (!W || !codes || !absmax) return LORA_ERR_INVALID_ARG;
  if (d_out <= 0 || d_in <= 0) return LORA_ERR_INVALID_ARG;
  if (d_in % kNf4Block != 0 || d_out % 4 != 0 || d_out > (1ll << 24) || d_in > (1ll << 24)) return LORA_ERR_UNSUPPORTED_SHAPE;
  if (!aligned16(W) || !aligned16(codes) || !aligned16(absmax)) return LORA_ERR_MISALIGNED;
  if (launch_nf4_quantize(static_cast<const __nv_bfloat16*>(W), d_out, d_in, static_cast<uint8_t*>(codes),
                          static_cast<float*>(absmax), static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  return LORA_OK;
}

int lora_nf4_dequantize(const void* W_codes, const void* W_absmax, int64_t d_out, int64_t d_in, void* W, void* stream) {
  if (!W || !W_codes || !W_absmax) return LORA_ERR_INVALID_ARG;
  if (d_out <= 0 || d_in <= 0) return LORA_ERR_INVALID_ARG;
  if (d_in % kNf4Block != 0 || d_out % 4 != 0 || d_out > (1ll << 24) || d_in > (1ll << 24)) return LORA_ERR_UNSUPPORTED_SHAPE;
  if (!aligned16(W) || !aligned16(W_codes) || !aligned16(W_absmax)) return LORA_ERR_MISALIGNED;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return LORA_ERR_CUDA;
  if (launch_nf4_dequantize(static_cast<const uint8_t*>(W_codes), static_cast<const float*>(W_absmax), d_out, d_in,
                            static_cast<__nv_bfloat16*>(W), sms, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  return LORA_OK;
}

int lora_linear_fwd_nf4(lora_plan_t* plan, const void* X, const void* W_codes, const void* W_absmax, const void* A,
                        const void* B, float scale, void* Y, void* w_scratch, void* stream) {
  if (plan == nullptr) return LORA_ERR_INVALID_ARG;
  if (plan->shape.T == 0) return LORA_OK;
  if (!X || !W_codes || !W_absmax || !A || !B || !Y) return LORA_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(W_codes) || !aligned16(W_absmax) || !aligned16(A) || !aligned16(B) || !aligned16(Y) ||
      !aligned16(w_scratch))
    return LORA_ERR_MISALIGNED;
  if (plan->shape.d_in % kNf4Block != 0 || plan->shape.d_out % 4 != 0) return LORA_ERR_UNSUPPORTED_SHAPE;
  DeviceGuard guard(plan->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (w_scratch != nullptr) {
    // expand once, then the bf16 path: every weight element is converted once per call instead of once per 256-token tile
    if (launch_nf4_dequantize(static_cast<const uint8_t*>(W_codes), static_cast<const float*>(W_absmax), plan->shape.d_out,
                              plan->shape.d_in, static_cast<__nv_bfloat16*>(w_scratch), plan->num_sms, st) != cudaSuccess)
      return LORA_ERR_CUDA;
    g_launches.fetch_add(1);
    return launch_fwd(plan, X, w_scratch, A, B, scale, Y, st);
  }
  const int rc = check_nf4(plan);
  if (rc != LORA_OK) return rc;
  return launch_fwd_nf4(plan, X, W_codes, W_absmax, A, B, scale, Y, st);
}

int lora_linear_bwd_nf4(lora_plan_t* plan, const void* dY, const void* X, const void* W_codes, const void* W_absmax,
                        const void* A, const void* B, float scale, void* dX, void* dA, void* dB, void* w_scratch,
                        void* stream) {
  if (plan == nullptr) return LORA_ERR_INVALID_ARG;
  if (!dA || !dB) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dA) || !aligned16(dB)) return LORA_ERR_MISALIGNED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  DeviceGuard guard(plan->device);
  if (plan->shape.T == 0) {
    if (plan->accumulate) return LORA_OK;
    if (cudaMemsetAsync(dA, 0, sizeof(float) * plan->shape.r * plan->shape.d_in, st) != cudaSuccess ||
        cudaMemsetAsync(dB, 0, sizeof(float) * plan->shape.d_out * plan->shape.r, st) != cudaSuccess)
      return LORA_ERR_CUDA;
    return LORA_OK;
  }
  if (!dY || !X || !W_codes || !W_absmax || !A || !B || !dX) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(X) || !aligned16(W_codes) || !aligned16(W_absmax) || !aligned16(A) || !aligned16(B) ||
      !aligned16(dX) || !aligned16(w_scratch))
    return LORA_ERR_MISALIGNED;
  plan->q_staged = false;
  if (plan->shape.d_in % kNf4Block != 0 || plan->shape.d_out % 4 != 0) return LORA_ERR_UNSUPPORTED_SHAPE;
  if (w_scratch != nullptr) {
    if (plan->workspace == nullptr || plan->workspace_bytes < plan->ws.total) return LORA_ERR_WORKSPACE;
    if (launch_nf4_dequantize(static_cast<const uint8_t*>(W_codes), static_cast<const float*>(W_absmax), plan->shape.d_out,
                              plan->shape.d_in, static_cast<__nv_bfloat16*>(w_scratch), plan->num_sms, st) != cudaSuccess)
      return LORA_ERR_CUDA;
    g_launches.fetch_add(1);
    int rc2 = launch_dx(plan, dY, w_scratch, A, B, scale, dX, st);
    if (rc2 == LORA_OK) rc2 = launch_da(plan, X, A, scale, dA, st);
    if (rc2 == LORA_OK) rc2 = launch_db(plan, dY, scale, dB, st);
    return rc2;
  }
  int rc = check_nf4(plan);
  if (rc != LORA_OK) return rc;
  rc = launch_dx_nf4(plan, dY, W_codes, W_absmax, A, B, scale, dX, st);
  if (rc == LORA_OK) rc = launch_da(plan, X, A, scale, dA, st);
  if (rc == LORA_OK) rc = launch_db(plan, dY, scale, dB, st);
  return rc;
}

int lora_dense_dw(lora_plan_t* plan, const void* dY, const void* X, void* dW, void* stream) {
  if (plan == nullptr || !dW) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dW)) return LORA_ERR_MISALIGNED;
  if (plan->num_sms < 2) return LORA_ERR_NO_DEVICE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  DeviceGuard guard(plan->device);
  if (plan->shape.T == 0)     // empty batch: the sum over tokens is empty
    return cudaMemsetAsync(dW, 0, sizeof(__nv_bfloat16) * plan->shape.d_out * plan->shape.d_in, st) == cudaSuccess
               ? LORA_OK : LORA_ERR_CUDA;
  if (!dY || !X) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(X)) return LORA_ERR_MISALIGNED;
  if (plan->cfg.dw_split_k > 1 && (plan->workspace == nullptr || plan->workspace_bytes < plan->ws.total))
    return LORA_ERR_WORKSPACE;
  return launch_dw(plan, dY, X, dW, st);
}

int lora_step_host_staging_bytes(const lora_shape_t* shape, size_t* bytes) {
  if (bytes == nullptr) return LORA_ERR_INVALID_ARG;
  const int rc = check_shape(shape);
  if (rc != LORA_OK) return rc;
  const size_t T = shape->T, di = shape->d_in, dout = shape->d_out, r = shape->r;
  size_t off = 0;
  off += align_up(T * di * 2, kAlign) * 2;      // X, dX
  off += align_up(T * dout * 2, kAlign) * 2;      // dY, Y
  off += align_up(r * di * 2, kAlign);          // A
  off += align_up(dout * r * 2, kAlign);          // B
  off += align_up(r * di * 4, kAlign);          // dA
  off += align_up(dout * r * 4, kAlign);          // dB
  *bytes = off;
  return LORA_OK;
}

int lora_linear_step_host(lora_plan_t* plan, const void* h_X, const void* W, const void* h_A, const void* h_B,
                          const void* h_dY, float scale, void* h_Y, void* h_dX, void* h_dA, void* h_dB, void* staging,
                          size_t staging_bytes, void* stream) {
  if (plan == nullptr) return LORA_ERR_INVALID_ARG;
  if (!h_X || !W || !h_A || !h_B || !h_dY || !h_Y || !h_dX || !h_dA || !h_dB || !staging) return LORA_ERR_INVALID_ARG;
  size_t need = 0;
  lora_step_host_staging_bytes(&plan->shape, &need);
  if (staging_bytes < need) return LORA_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(staging) & (kAlign - 1)) != 0) return LORA_ERR_MISALIGNED;
  const size_t T = plan->shape.T, di = plan->shape.d_in, dout = plan->shape.d_out, r = plan->shape.r;
  uint8_t* base = static_cast<uint8_t*>(staging);
  size_t off = 0;
  auto take = [&](size_t bytes) {
    uint8_t* p = base + off;
    off += align_up(bytes, kAlign);
    return p;
  };
  uint8_t* dXin = take(T * di * 2);
  uint8_t* ddX = take(T * di * 2);
  uint8_t* ddY = take(T * dout * 2);
  uint8_t* dYout = take(T * dout * 2);
  uint8_t* dAin = take(r * di * 2);
  uint8_t* dBin = take(dout * r * 2);
  uint8_t* ddA = take(r * di * 4);
  uint8_t* ddB = take(dout * r * 4);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  DeviceGuard guard(plan->device);
  bool ok = true;
  if (T > 0) {
    ok = ok && cudaMemcpyAsync(dXin, h_X, T * di * 2, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(ddY, h_dY, T * dout * 2, cudaMemcpyHostToDevice, st) == cudaSuccess;
  }
  ok = ok && cudaMemcpyAsync(dAin, h_A, r * di * 2, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(dBin, h_B, dout * r * 2, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (!ok) return LORA_ERR_CUDA;
  int rc = lora_linear_fwd(plan, dXin, W, dAin, dBin, scale, dYout, stream);
  if (rc != LORA_OK) return rc;
  rc = lora_linear_bwd(plan, ddY, dXin, W, dAin, dBin, scale, ddX, ddA, ddB, stream);
  if (rc != LORA_OK) return rc;
  if (T > 0) {
    ok = ok && cudaMemcpyAsync(h_Y, dYout, T * dout * 2, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h_dX, ddX, T * di * 2, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  }
  ok = ok && cudaMemcpyAsync(h_dA, ddA, r * di * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(h_dB, ddB, dout * r * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  return ok ? LORA_OK : LORA_ERR_CUDA;
}

int lora_last_device_status(lora_plan_t* plan, void* stream, int* code, char* msg, size_t n) {
  if (plan == nullptr || code == nullptr) return LORA_ERR_INVALID_ARG;
  DeviceGuard guard(plan->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(st) != cudaSuccess) return LORA_ERR_CUDA;
  unsigned word = 0;
  if (cudaMemcpy(&word, plan->d_status, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return LORA_ERR_CUDA;
  if (word == 0) {
    *code = LORA_OK;
    if (msg && n) std::snprintf(msg, n, "ok");
    return LORA_OK;
  }
  *code = LORA_ERR_DEVICE_TIMEOUT;
  static const char* what[] = {"",          "MMA waited for a TMA stage",        "TMA producer waited for a free stage",
                               "epilogue waited for the rank-r accumulator",     "MMA waited for the bf16 rank-r operand",
                               "epilogue waited for the accumulator",            "MMA waited for a drained accumulator",
                               "other wait"};
  if (msg && n) std::snprintf(msg, n, "device wait ran out: %s (CTA %u)", what[word & 7u], word >> 8);
  if (cudaMemset(plan->d_status, 0, 256) != cudaSuccess) return LORA_ERR_CUDA;
  return LORA_OK;
}

const char* lora_strerror(int code) {
  switch (code) {
    case LORA_OK: return "ok";
    case LORA_ERR_INVALID_ARG: return "invalid argument";
    case LORA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case LORA_ERR_MISALIGNED: return "pointer not sufficiently aligned";
    case LORA_ERR_WORKSPACE: return "workspace missing or too small";
    case LORA_ERR_CUDA: return "CUDA call failed";
    case LORA_ERR_DEVICE_TIMEOUT: return "a device-side wait ran out";
    case LORA_ERR_NO_DEVICE: return "no sm_100 CUDA device";
    default: return "unknown status";
  }
}

int64_t lora_launch_count(void) { return g_launches.load(); }

}  // extern "C"
