// C ABI of the LoRA projection layer: argument checks, the per-shape selector, plans, tensor maps and
// kernel launches.  See include/lora_linear.h for the contract of every entry point.
#include "../../include/lora_linear.h"

#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
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

// Streams of at most this many bytes are a few microseconds of work: they run on the smallest grid (one CTA per feature
// chunk of a gradient, one feature chunk for a side product), where nothing is summed across CTAs.
constexpr long long kTinyStreamBytes = 1 << 20;

// Grid of a side-product-only job (X A^T or dY B) that may use `ctas` CTAs: feature chunks x token chunks, no TMEM bound on
// the feature chunk.  Token slabs are independent, so ONE feature chunk is best whenever whole slabs spread evenly over the
// CTAs: every CTA sees all features of its slabs and writes the bf16 result itself.  When a CTA would get one or two very
// long slabs (few slabs, or wide matrices beside a narrow one in the same launch) the features are cut into 2, 4 or 8
// chunks, whose fp32 partials the last CTA to arrive for a slab adds up.  Cost of a candidate = bytes of its busiest CTA
// (+ 64 features' worth per slab for the arrival round trip when there are partials); ties go to fewer chunks.
struct SideGrid {
  int feat_chunk, n_feat, n_tok;
};

constexpr int kSideMaxChunks = 8;

SideGrid pick_side_grid(long long T, long long C, int ctas) {
  const int n_slabs = ceil_div(T, kGradSlab);
  const int nblk = ceil_div(C, 128);
  if (ctas < 1) ctas = 1;
  int best_nf = 1;
  double best_cost = 1e300;
  for (int nf = 1; nf <= kSideMaxChunks && nf <= nblk && nf <= ctas; nf *= 2) {
    const int fc = ceil_div(nblk, nf) * 128;
    const int n_feat = ceil_div(C, fc);
    int n_tok = ctas / n_feat;
    if (n_tok > n_slabs) n_tok = n_slabs;
    if (n_tok < 1) n_tok = 1;
    // a split pays per slab for the partial sums (fp32 write, fence, arrival counter, last-arriver sum): measured on the
    // 32768 x 4096 stream beside a 1024-wide one, 1 chunk x 3 slabs per CTA 58.0 us against 4 chunks x 9 slabs 64.0 us
    const double cost = static_cast<double>(ceil_div(n_slabs, n_tok)) * (fc + (n_feat > 1 ? 512 : 0));
    if (cost < best_cost * 0.97) {        // a split must pay for itself by a clear margin
      best_cost = cost;
      best_nf = nf;
    }
  }
  if (kTinyStreamBytes >= 2 * T * C) best_nf = 1;
  if (const char* f = std::getenv("LORA_PREPASS_NF")) {      // tuning knob
    const int v = std::atoi(f);
    if (v >= 1 && v <= kSideMaxChunks && v <= nblk) best_nf = v;
  }
  SideGrid g;
  g.feat_chunk = ceil_div(nblk, best_nf) * 128;
  g.n_feat = ceil_div(C, g.feat_chunk);
  g.n_tok = ctas / g.n_feat;
  if (g.n_tok > n_slabs) g.n_tok = n_slabs;
  if (g.n_tok < 1) g.n_tok = 1;
  return g;
}

// CTAs of a two-job side-product launch are shared out in proportion to the jobs' bytes
int side_pair_split(long long C0, long long C1, int num_sms) {
  int g0 = static_cast<int>((static_cast<double>(num_sms) * C0) / static_cast<double>(C0 + C1) + 0.5);
  if (g0 < 1) g0 = 1;
  if (g0 > num_sms - 1) g0 = num_sms - 1;
  return g0;
}

int check_shape(const lora_shape_t* s) {
  if (s == nullptr) return LORA_ERR_INVALID_ARG;
  if (s->T < 0 || s->d_in <= 0 || s->d_out <= 0 || s->r <= 0) return LORA_ERR_INVALID_ARG;
  if (s->T > (1ll << 30) || s->d_in > (1ll << 24) || s->d_out > (1ll << 24)) return LORA_ERR_UNSUPPORTED_SHAPE;
  if (s->d_in % 8 != 0 || s->d_out % 8 != 0) return LORA_ERR_UNSUPPORTED_SHAPE;
  if (s->r % 8 != 0 || s->r < 8 || s->r > 64) return LORA_ERR_UNSUPPORTED_SHAPE;
  return LORA_OK;
}

// `caps_in`: caps_in[cs] = CTAs of the streaming kernel resident at once in clusters of cs CTAs, cs = 1 .. 16 (asked from the
// device when a plan is created); nullptr: estimated from the SM count.
int select_config(const lora_shape_t* s, int num_sms, lora_kernel_config_t* c, const int* caps_in = nullptr) {
  const int rc = check_shape(s);
  if (rc != LORA_OK) return rc;
  if (num_sms <= 0 || c == nullptr) return LORA_ERR_INVALID_ARG;
  std::memset(c, 0, sizeof(*c));
  int caps[kGradMaxCluster + 1];
  if (caps_in != nullptr) {
    for (int i = 0; i <= kGradMaxCluster; ++i) caps[i] = caps_in[i];
  } else {
    grad_default_caps(num_sms, caps);
  }
  const long long T = s->T > 0 ? s->T : 1;
  c->block_m = kBlockM;
  c->block_k = kBlockK;
  c->r_pad = static_cast<int>((s->r + 15) / 16 * 16);
  c->fwd_block_n = pick_block_n(T, s->d_out, c->r_pad, num_sms);
  c->dx_block_n = pick_block_n(T, s->d_in, c->r_pad, num_sms);
  c->stages = 4;
  c->dx_stages = 4;
  // m-tiles per rasterisation band.  A weight that fits L2 several times over stays there whatever the order, so short bands
  // (activations fetched once, nothing else re-read) bring DRAM traffic down to the operands themselves: 8192 x 4096 x 4096,
  // forward GEMM 221 -> 172 MB per launch at the same 172 us.  A weight of L2's size needs tall bands to be reused at all.
  c->group_m = (2 * s->d_out * s->d_in <= (48ll << 20)) ? 2 : 8;
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
  // Backward owes three skinny products besides the dX GEMM: s (dY B)^T before it, and dA, dB, which need s (X A^T)^T.
  //  merged form (bwd_merged = 1): ONE launch computes dY B and X A^T side by side before the GEMM, ONE launch dA and dB
  //    after it.  Four passes over the activations (X and dY twice each), two launches, every CTA of a side product sees
  //    whole token slabs and every CTA of a gradient whole 128-feature blocks, so almost nothing is summed across CTAs.
  //  split form (bwd_merged = 0): dY B | GEMM | dA with X A^T riding along (da_with_p; for ranks above 32 its partial sums
  //    over feature chunks approach the size of the stream and X A^T gets its own pass) | dB: three passes, three launches.
  c->bwd_merged = 1;
  if (const char* f = std::getenv("LORA_FORCE_BWD_MERGED")) c->bwd_merged = std::atoi(f) != 0 ? 1 : 0;
  c->da_with_p = c->r_pad <= 32 ? 1 : 0;
  if (const char* f = std::getenv("LORA_FORCE_DA_WITH_P")) c->da_with_p = std::atoi(f) != 0 ? 1 : 0;
  const bool tiny_a = kTinyStreamBytes >= 2 * T * s->d_in, tiny_b = kTinyStreamBytes >= 2 * T * s->d_out;
  int caps1[kGradMaxCluster + 1] = {};                 // tiny streams: no clusters
  caps1[1] = caps[1];
  const GradGrid ga = grad_pick_grid(T, s->d_in, 0, c->r_pad, c->da_with_p != 0, false, tiny_a ? caps1 : caps);
  const GradGrid gb = grad_pick_grid(T, s->d_out, 0, c->r_pad, false, false, tiny_b ? caps1 : caps);
  c->grad_feat_chunk = ga.feat_chunk;
  c->grad_stages = ga.stages;
  c->db_stages = gb.stages;
  c->da_feat_chunks = ga.n_feat;
  c->da_token_chunks = ga.n_tok;
  c->db_feat_chunks = gb.n_feat;
  c->db_token_chunks = gb.n_tok;
  c->db_feat_chunk = gb.feat_chunk;
  {
    // dA without the side product (split form with da_with_p = 0, saved-P backward); dB with dY B riding along (saved-P
    // backward, split form); dA and dB side by side in one launch (merged form): common chunk width and cluster size
    const GradGrid gan = grad_pick_grid(T, s->d_in, 0, c->r_pad, false, false, tiny_a ? caps1 : caps);
    const GradGrid gbq = grad_pick_grid(T, s->d_out, 0, c->r_pad, true, true, tiny_b ? caps1 : caps);
    const GradGrid gp = grad_pick_grid(T, s->d_in, s->d_out, c->r_pad, false, false, (tiny_a && tiny_b) ? caps1 : caps);
    c->dan_feat_chunk = gan.feat_chunk;
    c->dan_feat_chunks = gan.n_feat;
    c->dan_token_chunks = gan.n_tok;
    c->dbq_feat_chunk = gbq.feat_chunk;
    c->dbq_feat_chunks = gbq.n_feat;
    c->dbq_token_chunks = gbq.n_tok;
    c->pair_feat_chunk = gp.feat_chunk;
    c->pair_feat_chunks = gp.n_feat;
    c->pair_token_chunks = gp.n_tok;
  }
  {  // Q = dY B pre-pass of the CTA-pair backward
    const SideGrid q = pick_side_grid(T, s->d_out, num_sms);
    c->q_feat_chunk = q.feat_chunk;
    c->q_feat_chunks = q.n_feat;
    c->q_token_chunks = q.n_tok;
    GradParams t{};
    t.with_p = 1;
    t.side_mn = 1;
    t.r_pad = c->r_pad;
    t.feat_chunk = q.feat_chunk;
    grad_set_ring(&t);
    c->q_stages = t.stages;
  }
  return LORA_OK;
}

// ------------------------------------------------------------------------------------------------
// backward workspace layout
// ------------------------------------------------------------------------------------------------
struct WsLayout {
  size_t qt, pt, q_part, p_part, count, split_part, total;
  int ld_t, n_slabs;
};

WsLayout ws_layout(const lora_shape_t& s, const lora_kernel_config_t& c) {
  WsLayout w;
  const long long T = s.T > 0 ? s.T : 1;
  w.ld_t = static_cast<int>(align_up(static_cast<size_t>(T), 64));
  w.n_slabs = ceil_div(T, kGradSlab);
  size_t off = 0;
  w.qt = off;       off += align_up(static_cast<size_t>(c.r_pad) * w.ld_t * 2, kAlign);
  w.pt = off;       off += align_up(static_cast<size_t>(c.r_pad) * w.ld_t * 2, kAlign);
  {
    // fp32 partials of a side product computed with more than one feature chunk: the side-only jobs use at most
    // kSideMaxChunks; the launches where it rides a gradient have one per feature chunk of that grid
    int q_chunks = c.dbq_feat_chunks > kSideMaxChunks ? c.dbq_feat_chunks : kSideMaxChunks;
    int p_chunks = c.da_feat_chunks > kSideMaxChunks ? c.da_feat_chunks : kSideMaxChunks;
    w.q_part = off;   off += align_up(static_cast<size_t>(q_chunks) * c.r_pad * w.ld_t * 4, kAlign);
    w.p_part = off;   off += align_up(static_cast<size_t>(p_chunks) * c.r_pad * w.ld_t * 4, kAlign);
  }
  w.count = off;    off += align_up(2 * static_cast<size_t>(w.n_slabs) * sizeof(int), kAlign);   // per-slab arrival counters, two jobs
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
  int caps[kGradMaxCluster + 1];   // caps[cs]: CTAs of the streaming kernel resident at once in clusters of cs CTAs
  bool counters_clean;   // the workspace's arrival counters are known to be zero
  bool p_saved;          // the workspace holds Pt = s (X A^T)^T of the last forward call
  float p_saved_scale;
  long long wait_limit;  // SM clock ticks after which a device-side spin gives up (lora_plan_set_wait_limit)
  size_t nf4_scratch_bytes;   // bytes behind the w_scratch of the Q+LoRA calls; 0 = the whole weight (lora_plan_set_nf4_scratch_bytes)
  // grouped projections (lora_plan_create_grouped): G projections that share X; shape.d_out is the sum of their widths
  int n_groups;          // 0: an ordinary plan
  long long group_off[5];   // first output column of every group, and the total
  struct GroupedWs {
    size_t qt, pt, part, count, total;    // Qt_all / Pt_all [G r, ld_t] bf16, partial-sum regions, counters
    size_t part_stride;                   // bytes of one job's partial-sum region
  } gws;
};

namespace {

// caps[cs] = CTAs of the streaming kernel resident at once in clusters of cs CTAs on `device` (current): asked once per
// device; a size the device refuses gets 0 and is never chosen.
void device_caps(int device, int num_sms, int* caps) {
  static std::mutex mu;
  static int table[64][kGradMaxCluster + 1];
  static bool ready[64] = {};
  std::lock_guard<std::mutex> lock(mu);
  if (device < 0 || device >= 64) {
    grad_device_caps(num_sms, caps);
    return;
  }
  if (!ready[device]) {
    grad_device_caps(num_sms, table[device]);
    ready[device] = true;
  }
  for (int i = 0; i <= kGradMaxCluster; ++i) caps[i] = table[device][i];
}

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

// The arrival counters of the side-product partials live in the caller's workspace.  Every launch leaves them at zero;
// they are cleared on `st` before the first launch after the workspace was registered (or after a wait ran out).
bool ensure_counters(lora_plan* pl, cudaStream_t st) {
  if (pl->counters_clean) return true;
  if (cudaMemsetAsync(static_cast<uint8_t*>(pl->workspace) + pl->ws.count, 0, 2 * static_cast<size_t>(pl->ws.n_slabs) * sizeof(int), st) !=
      cudaSuccess)
    return false;
  pl->counters_clean = true;
  return true;
}

// One side-product job: out_t = s (S side^T)^T as bf16 [r_pad, ld_t], S = X with side = A [r, C] (K-major) or S = dY with
// side = B [C, r] (MN-major).  Streams S once on at most `ctas` CTAs; `which` (0 / 1) picks the job's own partial-sum region
// and counter range, so that two jobs can run side by side.
struct SideJob {
  CUtensorMap tmS, tmSide;
  GradParams g;
};

bool fill_side_job(lora_plan* pl, const void* S, long long C, const void* side, bool side_mn, float scale, __nv_bfloat16* out_t,
                   int ctas, int which, SideJob* job) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  const WsLayout& w = pl->ws;
  bool ok = make_bf16_tmap(&job->tmS, S, C, s.T, C, 64, kGradSlab);
  if (side_mn) ok = ok && make_bf16_tmap(&job->tmSide, side, s.r, C, s.r, 64, 64);
  else ok = ok && make_bf16_tmap(&job->tmSide, side, C, s.r, C, 64, c.r_pad);
  if (!ok) return false;
  const SideGrid sg = pick_side_grid(s.T, C, ctas);
  GradParams g{};
  g.T = static_cast<int>(s.T);
  g.C = static_cast<int>(C);
  g.r = static_cast<int>(s.r);
  g.r_pad = c.r_pad;
  g.feat_chunk = sg.feat_chunk;
  g.n_feat_chunks = sg.n_feat;
  g.n_token_chunks = sg.n_tok;
  g.n_slabs = w.n_slabs;
  g.tmem_cols = grad_tmem_cols(sg.feat_chunk, c.r_pad, false, true);
  g.with_p = 1;
  g.side_mn = side_mn ? 1 : 0;
  g.do_out = 0;
  g.scale = scale;
  uint8_t* ws = static_cast<uint8_t*>(pl->workspace);
  g.p_part = reinterpret_cast<float*>(ws + (which == 0 ? w.q_part : w.p_part));
  g.side_count = reinterpret_cast<int*>(ws + w.count) + (which == 0 ? 0 : w.n_slabs);
  g.pt_out = out_t;
  g.ld_t = w.ld_t;
  g.status = pl->d_status;
  g.wait_limit = pl->wait_limit;
  job->g = g;
  return true;
}

// one side product alone (X A^T before a K-extended forward GEMM, dY B before the dX GEMM)
int launch_side_prepass(lora_plan* pl, const void* S, long long C, const void* side, bool side_mn, float scale,
                        __nv_bfloat16* out_t, cudaStream_t st) {
  SideJob j;
  if (!fill_side_job(pl, S, C, side, side_mn, scale, out_t, pl->num_sms, side_mn ? 0 : 1, &j)) return LORA_ERR_CUDA;
  if (j.g.n_feat_chunks > 1 && !ensure_counters(pl, st)) return LORA_ERR_CUDA;
  if (launch_grad(j.tmS, j.tmS, j.tmSide, j.g, st) != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  return LORA_OK;
}

// Qt = s (dY B)^T and Pt = s (X A^T)^T in ONE launch: the two jobs share the SMs in proportion to their bytes
int launch_side_pair(lora_plan* pl, const void* dY, const void* B, const void* X, const void* A, float scale, cudaStream_t st) {
  const lora_shape_t& s = pl->shape;
  const WsPtrs q = ws_ptrs(pl);
  const int g0 = side_pair_split(s.d_out, s.d_in, pl->num_sms);
  SideJob jq, jp;
  if (!fill_side_job(pl, dY, s.d_out, B, true, scale, q.qt, g0, 0, &jq) ||
      !fill_side_job(pl, X, s.d_in, A, false, scale, q.pt, pl->num_sms - g0, 1, &jp))
    return LORA_ERR_CUDA;
  if ((jq.g.n_feat_chunks > 1 || jp.g.n_feat_chunks > 1) && !ensure_counters(pl, st)) return LORA_ERR_CUDA;
  GradJobDesc jobs[2];
  jobs[0].tmS = jobs[0].tmR = jq.tmS;
  jobs[0].tmSide = jq.tmSide;
  jobs[0].p = jq.g;
  jobs[1].tmS = jobs[1].tmR = jp.tmS;
  jobs[1].tmSide = jp.tmSide;
  jobs[1].p = jp.g;
  if (launch_grad_jobs(jobs, 2, st) != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  return LORA_OK;
}

// A window of the GEMM's output columns: columns [off, off + n) of Y (forward: output features, W = the n weight rows of the
// window, row pitch d_in) or of dX (backward: input features, W = the window's n columns of every weight row, row pitch n).
// The banded Q+LoRA calls run one GEMM launch per window; `first` = the launch that also runs the skinny pre-pass.
struct ColWindow {
  long long off, n;
  bool first;
};

int launch_fwd(lora_plan* pl, const void* X, const void* W, const void* A, const void* B, float scale, void* Y,
               cudaStream_t st, const ColWindow* win = nullptr) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  const bool pair = c.cta_group == 2;
  const bool ext = pair && c.fwd_ext != 0;
  const bool have_ws = pl->workspace != nullptr && pl->workspace_bytes >= pl->ws.total;
  if (ext && !have_ws) return LORA_ERR_WORKSPACE;
  __nv_bfloat16* pt = have_ws ? ws_ptrs(pl).pt : nullptr;
  if (ext && (win == nullptr || win->first)) {
    const int rc = launch_side_prepass(pl, X, s.d_in, A, false, scale, pt, st);   // Pt = s (X A^T)^T
    if (rc != LORA_OK) return rc;
  }
  const long long n_out = win ? win->n : s.d_out;            // output columns of this launch
  if (win) {                                                   // W already points at the window's rows
    B = static_cast<const __nv_bfloat16*>(B) + win->off * s.r;
    Y = static_cast<__nv_bfloat16*>(Y) + win->off;
  }
  const int half = (c.fwd_block_n + c.r_pad) / 2;
  CUtensorMap tmX, tmW, tmW1, tmA, tmB, tmY;
  bool ok = make_bf16_tmap(&tmX, X, s.d_in, s.T, s.d_in, 64, kBlockM);
  ok = ok && make_bf16_tmap(&tmW, W, s.d_in, n_out, s.d_in, 64, ext ? c.fwd_block_n / 2 : pair ? half : c.fwd_block_n);
  if (pair && !ext) ok = ok && make_bf16_tmap(&tmW1, W, s.d_in, n_out, s.d_in, 64, c.fwd_block_n - half);
  if (ext) ok = ok && make_bf16_tmap(&tmA, pt, s.T, c.r_pad, pl->ws.ld_t, 64, c.r_pad);
  else ok = ok && make_bf16_tmap(&tmA, A, s.d_in, s.r, s.d_in, 64, c.r_pad);
  ok = ok && make_bf16_tmap(&tmB, B, s.r, n_out, s.r, 64, pair ? c.fwd_block_n / 2 : c.fwd_block_n);
  ok = ok && make_bf16_tmap(&tmY, Y, n_out, s.T, s.d_out, 64, kBlockM);
  if (!ok) return LORA_ERR_CUDA;
  GemmParams p{};
  p.out = static_cast<__nv_bfloat16*>(Y);
  p.ld_out = static_cast<int>(s.d_out);
  p.M = static_cast<int>(s.T);
  p.N = static_cast<int>(n_out);
  p.K = static_cast<int>(s.d_in);
  p.r_pad = c.r_pad;
  p.block_n = c.fwd_block_n;
  p.tiles_m = ceil_div(s.T, c.block_m);
  p.tiles_n = ceil_div(n_out, c.fwd_block_n);
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
    p.tail_parts = 1;
  if (win && p.split_k > 1) return LORA_ERR_UNSUPPORTED_SHAPE;   // the split-K reduction writes whole contiguous outputs
  int fwd_ctas = c.fwd_ctas;
  if (win && pair && fwd_ctas > 2 * p.num_tiles) fwd_ctas = 2 * p.num_tiles;
  const cudaError_t le = ext    ? launch_gemm_pair_fwd_ext(tmX, tmW, tmA, tmB, tmY, p, fwd_ctas, st)
                         : pair ? launch_gemm_pair_fwd(tmX, tmW, tmW1, tmA, tmB, tmY, p, fwd_ctas, st)
                                : launch_gemm_fwd(tmX, tmW, tmA, tmB, tmY, p, fwd_ctas, st);
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
              cudaStream_t st, int ctas_override = 0, const ColWindow* win = nullptr) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  const WsLayout& w = pl->ws;
  const WsPtrs q = ws_ptrs(pl);
  __nv_bfloat16* qt = q.qt;
  const long long n_in = win ? win->n : s.d_in;              // input features (columns of dX) of this launch
  const long long ld_w = win ? win->n : s.d_in;              // a window's weight columns are stored densely
  if (win) {
    A = static_cast<const __nv_bfloat16*>(A) + win->off;
    dX = static_cast<__nv_bfloat16*>(dX) + win->off;
  }
  if (c.cta_group == 2 && !pl->q_ready && (win == nullptr || win->first)) {
    // ---- pre-pass: Qt = s (dY B)^T, dY streamed once by the skinny kernel (side product only) ----
    const int rc = launch_side_prepass(pl, dY, s.d_out, B, true, scale, qt, st);
    if (rc != LORA_OK) return rc;
  }
  {
    CUtensorMap tmdY, tmW, tmB, tmA, tmdX;
    bool ok = make_bf16_tmap(&tmdY, dY, s.d_out, s.T, s.d_out, 64, kBlockM);
    ok = ok && make_bf16_tmap(&tmW, W, n_in, s.d_out, ld_w, 64, 64);
    const bool pair = c.cta_group == 2;
    if (pair) ok = ok && make_bf16_tmap(&tmB, qt, s.T, c.r_pad, w.ld_t, 64, c.r_pad);   // Qt from the pre-pass above
    else ok = ok && make_bf16_tmap(&tmB, B, s.r, s.d_out, s.r, 64, 64);
    ok = ok && make_bf16_tmap(&tmA, A, n_in, s.r, s.d_in, 64, c.r_pad);
    ok = ok && make_bf16_tmap(&tmdX, dX, n_in, s.T, s.d_in, 64, kBlockM);
    if (!ok) return LORA_ERR_CUDA;
    GemmParams p{};
    p.out = static_cast<__nv_bfloat16*>(dX);
    p.ld_out = static_cast<int>(s.d_in);
    p.M = static_cast<int>(s.T);
    p.N = static_cast<int>(n_in);
    p.K = static_cast<int>(s.d_out);
    p.r_pad = c.r_pad;
    p.block_n = c.dx_block_n;
    p.tiles_m = ceil_div(s.T, c.block_m);
    p.tiles_n = ceil_div(n_in, c.dx_block_n);
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
    p.tail_parts = 1;
    if (win && (p.split_k > 1 || !pair)) return LORA_ERR_UNSUPPORTED_SHAPE;
    int ctas = ctas_override > 0 ? ctas_override : c.dx_ctas;
    if (win && ctas > 2 * p.num_tiles) ctas = 2 * p.num_tiles;
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

// ---- gradient jobs: dA = Qt-contraction over X, dB = Pt-contraction over dY ----
struct GradJob {
  CUtensorMap tmS, tmR, tmSide;
  GradParams g;
};

// dA over X with second factor Qt; with_p: X A^T rides along and Pt = s (X A^T)^T is left in the workspace.
// (feat_chunk, n_feat, n_tok) = grid of the launch this job belongs to (its own feature chunks are derived from feat_chunk).
bool fill_da_job(lora_plan* pl, const void* X, const void* A, float scale, void* dA, bool with_p, int feat_chunk, int n_tok,
                 GradJob* job) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  const WsLayout& w = pl->ws;
  const WsPtrs q = ws_ptrs(pl);
  bool ok = make_bf16_tmap(&job->tmS, X, s.d_in, s.T, s.d_in, 64, kGradSlab);
  ok = ok && make_bf16_tmap(&job->tmR, q.qt, s.T, c.r_pad, w.ld_t, 64, c.r_pad);
  ok = ok && make_bf16_tmap(&job->tmSide, A, s.d_in, s.r, s.d_in, 64, c.r_pad);
  if (!ok) return false;
  GradParams g{};
  g.T = static_cast<int>(s.T);
  g.C = static_cast<int>(s.d_in);
  g.r = static_cast<int>(s.r);
  g.r_pad = c.r_pad;
  g.feat_chunk = feat_chunk;
  g.n_feat_chunks = ceil_div(s.d_in, feat_chunk);
  g.n_token_chunks = n_tok;
  g.n_slabs = w.n_slabs;
  g.tmem_cols = grad_tmem_cols(feat_chunk, c.r_pad, true, with_p);
  g.with_p = with_p ? 1 : 0;
  g.side_mn = 0;
  g.do_out = 1;
  g.out_is_da = 1;
  g.accumulate = pl->accumulate ? 1 : 0;
  g.scale = scale;
  g.out = static_cast<float*>(dA);
  g.p_part = reinterpret_cast<float*>(q.base + w.p_part);
  g.side_count = reinterpret_cast<int*>(q.base + w.count) + w.n_slabs;
  g.pt_out = q.pt;
  g.ld_t = w.ld_t;
  g.status = pl->d_status;
  g.wait_limit = pl->wait_limit;
  job->g = g;
  return true;
}

// dB over dY with second factor Pt; B_for_q: dY B rides along and Qt = s (dY B)^T is left in the workspace (saved-P backward)
bool fill_db_job(lora_plan* pl, const void* dY, float scale, void* dB, const void* B_for_q, int feat_chunk, int n_tok,
                 GradJob* job) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  const WsLayout& w = pl->ws;
  const WsPtrs q = ws_ptrs(pl);
  const bool with_q = B_for_q != nullptr;
  bool ok = make_bf16_tmap(&job->tmS, dY, s.d_out, s.T, s.d_out, 64, kGradSlab);
  ok = ok && make_bf16_tmap(&job->tmR, q.pt, s.T, c.r_pad, w.ld_t, 64, c.r_pad);
  if (with_q) ok = ok && make_bf16_tmap(&job->tmSide, B_for_q, s.r, s.d_out, s.r, 64, 64);
  else job->tmSide = job->tmR;
  if (!ok) return false;
  GradParams g{};
  g.T = static_cast<int>(s.T);
  g.C = static_cast<int>(s.d_out);
  g.r = static_cast<int>(s.r);
  g.r_pad = c.r_pad;
  g.feat_chunk = feat_chunk;
  g.n_feat_chunks = ceil_div(s.d_out, feat_chunk);
  g.n_token_chunks = n_tok;
  g.n_slabs = w.n_slabs;
  g.tmem_cols = grad_tmem_cols(feat_chunk, c.r_pad, true, with_q);
  g.with_p = with_q ? 1 : 0;
  g.side_mn = with_q ? 1 : 0;
  g.do_out = 1;
  g.out_is_da = 0;
  g.accumulate = pl->accumulate ? 1 : 0;
  g.scale = scale;
  g.out = static_cast<float*>(dB);
  g.p_part = with_q ? reinterpret_cast<float*>(q.base + w.q_part) : nullptr;
  g.side_count = reinterpret_cast<int*>(q.base + w.count);
  g.pt_out = with_q ? q.qt : nullptr;
  g.ld_t = w.ld_t;
  g.status = pl->d_status;
  g.wait_limit = pl->wait_limit;
  job->g = g;
  return true;
}

int launch_da(lora_plan* pl, const void* X, const void* A, float scale, void* dA, cudaStream_t st, bool with_p) {
  const lora_kernel_config_t& c = pl->cfg;
  const bool cfg_grid = with_p == (c.da_with_p != 0);       // the plan's default dA launch, else the form without X A^T
  if (with_p && !cfg_grid) return LORA_ERR_INVALID_ARG;     // only the plan's own with-side grid is sized for TMEM and scratch
  GradJob j;
  if (!fill_da_job(pl, X, A, scale, dA, with_p, cfg_grid ? c.grad_feat_chunk : c.dan_feat_chunk,
                   cfg_grid ? c.da_token_chunks : c.dan_token_chunks, &j))
    return LORA_ERR_CUDA;
  if (with_p && j.g.n_feat_chunks > 1 && !ensure_counters(pl, st)) return LORA_ERR_CUDA;
  if (launch_grad(j.tmS, j.tmR, j.tmSide, j.g, st) != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  return LORA_OK;
}

int launch_db(lora_plan* pl, const void* dY, float scale, void* dB, cudaStream_t st, const void* B_for_q = nullptr) {
  const lora_kernel_config_t& c = pl->cfg;
  const bool with_q = B_for_q != nullptr;
  GradJob j;
  if (!fill_db_job(pl, dY, scale, dB, B_for_q, with_q ? c.dbq_feat_chunk : c.db_feat_chunk,
                   with_q ? c.dbq_token_chunks : c.db_token_chunks, &j))
    return LORA_ERR_CUDA;
  if (with_q && j.g.n_feat_chunks > 1 && !ensure_counters(pl, st)) return LORA_ERR_CUDA;
  if (launch_grad(j.tmS, j.tmR, j.tmSide, j.g, st) != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  return LORA_OK;
}

// dA and dB in ONE launch (both second factors are ready): the feature chunks of X and of dY side by side
int launch_grad_pair(lora_plan* pl, const void* X, const void* dY, const void* A, float scale, void* dA, void* dB,
                     cudaStream_t st) {
  const lora_kernel_config_t& c = pl->cfg;
  GradJob ja, jb;
  if (!fill_da_job(pl, X, A, scale, dA, false, c.pair_feat_chunk, c.pair_token_chunks, &ja) ||
      !fill_db_job(pl, dY, scale, dB, nullptr, c.pair_feat_chunk, c.pair_token_chunks, &jb))
    return LORA_ERR_CUDA;
  GradJobDesc jobs[2];
  jobs[0].tmS = ja.tmS;
  jobs[0].tmR = ja.tmR;
  jobs[0].tmSide = ja.tmSide;
  jobs[0].p = ja.g;
  jobs[1].tmS = jb.tmS;
  jobs[1].tmR = jb.tmR;
  jobs[1].tmSide = jb.tmSide;
  jobs[1].p = jb.g;
  if (launch_grad_jobs(jobs, 2, st) != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  return LORA_OK;
}

// ---- dA stage of the plain backward: dA, and Pt = s (X A^T)^T left for the dB launch.  X A^T rides the dA launch or,
//      for large ranks, comes from its own skinny pass over X first (cfg.da_with_p) ----
int launch_da_stage(lora_plan* pl, const void* X, const void* A, float scale, void* dA, cudaStream_t st) {
  const bool with_p = pl->cfg.da_with_p != 0;
  int rc = LORA_OK;
  if (!with_p) rc = launch_side_prepass(pl, X, pl->shape.d_in, A, false, scale, ws_ptrs(pl).pt, st);
  if (rc == LORA_OK) rc = launch_da(pl, X, A, scale, dA, st, with_p);
  return rc;
}

// ---- everything of the backward pass that follows the dX GEMM: dA and dB (Qt is in the workspace; Pt only if p_ready) ----
int launch_adapter_grads(lora_plan* pl, const void* dY, const void* X, const void* A, float scale, void* dA, void* dB,
                         bool p_ready, cudaStream_t st) {
  int rc = LORA_OK;
  if (pl->cfg.bwd_merged) {
    if (!p_ready) rc = launch_side_prepass(pl, X, pl->shape.d_in, A, false, scale, ws_ptrs(pl).pt, st);
    if (rc == LORA_OK) rc = launch_grad_pair(pl, X, dY, A, scale, dA, dB, st);
    return rc;
  }
  if (p_ready) rc = launch_da(pl, X, A, scale, dA, st, false);
  else rc = launch_da_stage(pl, X, A, scale, dA, st);
  if (rc == LORA_OK) rc = launch_db(pl, dY, scale, dB, st);
  return rc;
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
    p.tail_parts = 1;
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
  if (!pl->q_ready) {
    const int rc = launch_side_prepass(pl, dY, s.d_out, B, true, scale, qt, st);   // Qt = s (dY B)^T
    if (rc != LORA_OK) return rc;
  }
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
    p.tail_parts = 1;
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

// ---- Q+LoRA with a scratch buffer smaller than the weight: the weight is expanded band by band ----
// Forward: bands of output features (weight rows), each a whole number of n-tiles; backward: bands of input features (weight
// columns).  Every band is expanded into the scratch buffer and fed to the bf16 GEMM restricted to that band's output
// columns, so each weight element is still converted once per call and the tiles, their k-order and hence the results are
// those of the whole-weight scratch form.  A band of a few MB stays in L2 between its expansion and the GEMM that reads it.
size_t nf4_full_bytes(const lora_plan* pl) { return static_cast<size_t>(pl->shape.d_out) * pl->shape.d_in * 2; }

size_t nf4_min_bytes(const lora_plan* pl) {
  const size_t f = static_cast<size_t>(pl->cfg.fwd_block_n) * pl->shape.d_in * 2;
  const size_t b = static_cast<size_t>(pl->cfg.dx_block_n) * pl->shape.d_out * 2;
  return f > b ? f : b;
}

bool nf4_banded(const lora_plan* pl) { return pl->nf4_scratch_bytes != 0 && pl->nf4_scratch_bytes < nf4_full_bytes(pl); }

// n-tiles per band: as many as fit `max_tiles`, among those the count with the fewest modelled waves over the whole GEMM (every
// band ends in a partly filled wave of CTA pairs and pays one expansion launch)
long long nf4_band_tiles(long long tiles_m, long long tiles_n, long long max_tiles, int pairs) {
  if (max_tiles >= tiles_n) return tiles_n;
  long long best = 1;
  double best_cost = 0;
  for (long long k = 1; k <= max_tiles; ++k) {
    const long long full = tiles_n / k, rest = tiles_n - full * k;
    double cost = static_cast<double>(full) * (static_cast<double>(ceil_div(tiles_m * k, pairs)) + 0.3);
    if (rest) cost += static_cast<double>(ceil_div(tiles_m * rest, pairs)) + 0.3;
    if (k == 1 || cost <= best_cost) {
      best = k;
      best_cost = cost;
    }
  }
  return best;
}

int check_nf4_banded(const lora_plan* pl) {
  const lora_kernel_config_t& c = pl->cfg;
  if (c.cta_group != 2 || c.split_k != 1 || c.dx_split_k != 1) return LORA_ERR_UNSUPPORTED_SHAPE;   // needs the whole-weight scratch
  if (pl->nf4_scratch_bytes < nf4_min_bytes(pl)) return LORA_ERR_WORKSPACE;
  if (pl->workspace == nullptr || pl->workspace_bytes < pl->ws.total) return LORA_ERR_WORKSPACE;
  return LORA_OK;
}

int launch_fwd_nf4_banded(lora_plan* pl, const void* X, const void* codes, const void* absmax, const void* A, const void* B,
                          float scale, void* Y, void* scratch, cudaStream_t st) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  const long long bn = c.fwd_block_n;
  const long long max_tiles = static_cast<long long>(pl->nf4_scratch_bytes / (2 * static_cast<size_t>(s.d_in))) / bn;
  const long long rows = bn * nf4_band_tiles(ceil_div(s.T, c.block_m), ceil_div(s.d_out, bn), max_tiles, pl->num_sms / 2);
  for (long long off = 0; off < s.d_out; off += rows) {
    const long long n = s.d_out - off < rows ? s.d_out - off : rows;
    if (launch_nf4_dequantize_window(static_cast<const uint8_t*>(codes), static_cast<const float*>(absmax), s.d_out, s.d_in, off,
                                     n, 0, s.d_in, static_cast<__nv_bfloat16*>(scratch), s.d_in, pl->num_sms, st) != cudaSuccess)
      return LORA_ERR_CUDA;
    g_launches.fetch_add(1);
    const ColWindow win{off, n, off == 0};
    const int rc = launch_fwd(pl, X, scratch, A, B, scale, Y, st, &win);
    if (rc != LORA_OK) return rc;
  }
  return LORA_OK;
}

int launch_dx_nf4_banded(lora_plan* pl, const void* dY, const void* codes, const void* absmax, const void* A, const void* B,
                         float scale, void* dX, void* scratch, cudaStream_t st) {
  const lora_shape_t& s = pl->shape;
  const lora_kernel_config_t& c = pl->cfg;
  const long long bn = c.dx_block_n;
  const long long max_tiles = static_cast<long long>(pl->nf4_scratch_bytes / (2 * static_cast<size_t>(s.d_out))) / bn;
  const long long cols = bn * nf4_band_tiles(ceil_div(s.T, c.block_m), ceil_div(s.d_in, bn), max_tiles, pl->num_sms / 2);
  for (long long off = 0; off < s.d_in; off += cols) {
    const long long n = s.d_in - off < cols ? s.d_in - off : cols;
    if (launch_nf4_dequantize_window(static_cast<const uint8_t*>(codes), static_cast<const float*>(absmax), s.d_out, s.d_in, 0,
                                     s.d_out, off, n, static_cast<__nv_bfloat16*>(scratch), n, pl->num_sms, st) != cudaSuccess)
      return LORA_ERR_CUDA;
    g_launches.fetch_add(1);
    const ColWindow win{off, n, off == 0};
    const int rc = launch_dx(pl, dY, scratch, A, B, scale, dX, st, 0, &win);
    if (rc != LORA_OK) return rc;
  }
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
    p.tail_parts = 1;
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

// ------------------------------------------------------------------------------------------------
// grouped projections: several projections that consume the same X (q/k/v, gate/up) as ONE forward GEMM over the
// concatenated output columns, ONE dX GEMM over the concatenated contraction, and two skinny launches
// ------------------------------------------------------------------------------------------------
constexpr int kGroupRowsPerJob = 64;       // rank rows one streaming job handles (its r_pad)

// generic side-product job: out_t[rows, T] = scale (S side^T)^T for `rows` adapter rows
bool build_side_job(lora_plan* pl, const void* S, long long C, long long pitch, const void* side, bool side_mn, long long side_pitch,
                    int rows, float scale, __nv_bfloat16* out_t, float* part, int* count, int ctas, GradJobDesc* job) {
  const long long T = pl->shape.T;
  bool ok = make_bf16_tmap(&job->tmS, S, C, T, pitch, 64, kGradSlab);
  if (side_mn) ok = ok && make_bf16_tmap(&job->tmSide, side, rows, C, side_pitch, 64, 64);
  else ok = ok && make_bf16_tmap(&job->tmSide, side, C, rows, side_pitch, 64, rows);
  if (!ok) return false;
  job->tmR = job->tmS;
  const SideGrid sg = pick_side_grid(T, C, ctas);
  GradParams g{};
  g.T = static_cast<int>(T);
  g.C = static_cast<int>(C);
  g.r = rows;
  g.r_pad = rows;
  g.feat_chunk = sg.feat_chunk;
  g.n_feat_chunks = sg.n_feat;
  g.n_token_chunks = sg.n_tok;
  g.n_slabs = pl->ws.n_slabs;
  g.tmem_cols = grad_tmem_cols(sg.feat_chunk, rows, false, true);
  g.with_p = 1;
  g.side_mn = side_mn ? 1 : 0;
  g.do_out = 0;
  g.scale = scale;
  g.p_part = part;
  g.side_count = count;
  g.pt_out = out_t;
  g.ld_t = pl->ws.ld_t;
  g.status = pl->d_status;
  g.wait_limit = pl->wait_limit;
  job->p = g;
  return true;
}

// generic gradient job: out = S^T Rt^T over the tokens, Rt [rows, T]
bool build_grad_job(lora_plan* pl, const void* S, long long C, long long pitch, const __nv_bfloat16* Rt, int rows, void* out,
                    bool out_is_da, int feat_chunk, int n_tok, GradJobDesc* job) {
  const long long T = pl->shape.T;
  bool ok = make_bf16_tmap(&job->tmS, S, C, T, pitch, 64, kGradSlab);
  ok = ok && make_bf16_tmap(&job->tmR, Rt, T, rows, pl->ws.ld_t, 64, rows);
  if (!ok) return false;
  job->tmSide = job->tmR;
  GradParams g{};
  g.T = static_cast<int>(T);
  g.C = static_cast<int>(C);
  g.r = rows;
  g.r_pad = rows;
  g.feat_chunk = feat_chunk;
  g.n_feat_chunks = ceil_div(C, feat_chunk);
  g.n_token_chunks = n_tok;
  g.n_slabs = pl->ws.n_slabs;
  g.tmem_cols = grad_tmem_cols(feat_chunk, rows, true, false);
  g.do_out = 1;
  g.out_is_da = out_is_da ? 1 : 0;
  g.accumulate = pl->accumulate ? 1 : 0;
  g.scale = 1.f;
  g.out = static_cast<float*>(out);
  g.ld_t = pl->ws.ld_t;
  g.status = pl->d_status;
  g.wait_limit = pl->wait_limit;
  job->p = g;
  return true;
}

// the side-product jobs of a grouped launch: [G jobs dY_g B_g ->] Qt rows of group g, and X A_cat^T in chunks of at most 64
// adapter rows -> Pt rows; CTAs are shared out in proportion to the bytes each job streams
int launch_grouped_sides(lora_plan* pl, const void* dY, const void* B, const void* X, const void* A, float scale, bool with_q,
                         cudaStream_t st) {
  const int G = pl->n_groups;
  const long long r = pl->shape.r, D = pl->shape.d_out, d_in = pl->shape.d_in, R = G * r;
  uint8_t* ws = static_cast<uint8_t*>(pl->workspace);
  __nv_bfloat16* qt = reinterpret_cast<__nv_bfloat16*>(ws + pl->gws.qt);
  __nv_bfloat16* pt = reinterpret_cast<__nv_bfloat16*>(ws + pl->gws.pt);
  const int ld_t = pl->ws.ld_t;
  const int n_p = ceil_div(R, kGroupRowsPerJob);
  const int n_jobs = (with_q ? G : 0) + n_p;
  double bytes = 0;
  for (int g = 0; g < G && with_q; ++g) bytes += static_cast<double>(pl->group_off[g + 1] - pl->group_off[g]);
  bytes += static_cast<double>(n_p) * d_in;
  GradJobDesc jobs[kGradMaxJobs];
  int j = 0, left = pl->num_sms;
  auto share = [&](long long C, int jobs_left) {
    int c = static_cast<int>(pl->num_sms * (static_cast<double>(C) / bytes) + 0.5);
    if (c < 1) c = 1;
    if (c > left - (jobs_left - 1)) c = left - (jobs_left - 1);
    left -= c;
    return c;
  };
  bool partials = false;
  for (int g = 0; g < G && with_q; ++g, ++j) {
    const long long off = pl->group_off[g], dg = pl->group_off[g + 1] - off;
    if (!build_side_job(pl, static_cast<const __nv_bfloat16*>(dY) + off, dg, D, static_cast<const __nv_bfloat16*>(B) + off * r, true, r,
                        static_cast<int>(r), scale, qt + static_cast<size_t>(g) * r * ld_t,
                        reinterpret_cast<float*>(ws + pl->gws.part + j * pl->gws.part_stride),
                        reinterpret_cast<int*>(ws + pl->gws.count) + j * pl->ws.n_slabs, share(dg, n_jobs - j), &jobs[j]))
      return LORA_ERR_CUDA;
    partials = partials || jobs[j].p.n_feat_chunks > 1;
  }
  for (int c = 0; c < n_p; ++c, ++j) {
    const long long row0 = static_cast<long long>(c) * kGroupRowsPerJob;
    const int rows = static_cast<int>(R - row0 < kGroupRowsPerJob ? R - row0 : kGroupRowsPerJob);
    if (!build_side_job(pl, X, d_in, d_in, static_cast<const __nv_bfloat16*>(A) + row0 * d_in, false, d_in, rows, scale,
                        pt + static_cast<size_t>(row0) * ld_t, reinterpret_cast<float*>(ws + pl->gws.part + j * pl->gws.part_stride),
                        reinterpret_cast<int*>(ws + pl->gws.count) + j * pl->ws.n_slabs, share(d_in, n_jobs - j), &jobs[j]))
      return LORA_ERR_CUDA;
    partials = partials || jobs[j].p.n_feat_chunks > 1;
  }
  if (partials && !pl->counters_clean) {
    if (cudaMemsetAsync(ws + pl->gws.count, 0, static_cast<size_t>(kGradMaxJobs) * pl->ws.n_slabs * sizeof(int), st) != cudaSuccess)
      return LORA_ERR_CUDA;
    pl->counters_clean = true;
  }
  if (launch_grad_jobs(jobs, n_jobs, st) != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  return LORA_OK;
}

// dA_cat (chunks of at most 64 adapter rows over X) and dB_g (every group over its columns of dY) in ONE launch
int launch_grouped_grads(lora_plan* pl, const void* dY, const void* X, void* dA, void* dB, cudaStream_t st) {
  const int G = pl->n_groups;
  const long long r = pl->shape.r, D = pl->shape.d_out, d_in = pl->shape.d_in, R = G * r;
  uint8_t* ws = static_cast<uint8_t*>(pl->workspace);
  const __nv_bfloat16* qt = reinterpret_cast<const __nv_bfloat16*>(ws + pl->gws.qt);
  const __nv_bfloat16* pt = reinterpret_cast<const __nv_bfloat16*>(ws + pl->gws.pt);
  const int ld_t = pl->ws.ld_t;
  const int n_a = ceil_div(R, kGroupRowsPerJob);
  long long C[kGradMaxJobs];
  int n_jobs = 0;
  for (int c = 0; c < n_a; ++c) C[n_jobs++] = d_in;
  for (int g = 0; g < G; ++g) C[n_jobs++] = pl->group_off[g + 1] - pl->group_off[g];
  const GradGrid gg = grad_pick_grid_jobs(pl->shape.T, C, n_jobs, kGroupRowsPerJob, false, false, pl->caps);
  GradJobDesc jobs[kGradMaxJobs];
  int j = 0;
  for (int c = 0; c < n_a; ++c, ++j) {
    const long long row0 = static_cast<long long>(c) * kGroupRowsPerJob;
    const int rows = static_cast<int>(R - row0 < kGroupRowsPerJob ? R - row0 : kGroupRowsPerJob);
    if (!build_grad_job(pl, X, d_in, d_in, qt + static_cast<size_t>(row0) * ld_t, rows, static_cast<float*>(dA) + row0 * d_in, true,
                        gg.feat_chunk, gg.n_tok, &jobs[j]))
      return LORA_ERR_CUDA;
  }
  for (int g = 0; g < G; ++g, ++j) {
    const long long off = pl->group_off[g], dg = pl->group_off[g + 1] - off;
    if (!build_grad_job(pl, static_cast<const __nv_bfloat16*>(dY) + off, dg, D, pt + static_cast<size_t>(g) * r * ld_t, static_cast<int>(r),
                        static_cast<float*>(dB) + off * r, false, gg.feat_chunk, gg.n_tok, &jobs[j]))
      return LORA_ERR_CUDA;
  }
  if (launch_grad_jobs(jobs, n_jobs, st) != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  return LORA_OK;
}

// forward GEMM over the concatenated output columns; the rank-r k-block of a tile takes its group's rows of s (X A^T)^T
int launch_grouped_fwd_gemm(lora_plan* pl, const void* X, const void* W, const void* B, float scale, void* Y, cudaStream_t st) {
  const lora_shape_t& s = pl->shape;
  const int pairs = pl->num_sms / 2, bn = 256, r = static_cast<int>(s.r);
  uint8_t* ws = static_cast<uint8_t*>(pl->workspace);
  CUtensorMap tmX, tmW, tmPt, tmB, tmY;
  bool ok = make_bf16_tmap(&tmX, X, s.d_in, s.T, s.d_in, 64, kBlockM);
  ok = ok && make_bf16_tmap(&tmW, W, s.d_in, s.d_out, s.d_in, 64, bn / 2);
  ok = ok && make_bf16_tmap(&tmPt, ws + pl->gws.pt, s.T, pl->n_groups * r, pl->ws.ld_t, 64, r);
  ok = ok && make_bf16_tmap(&tmB, B, s.r, s.d_out, s.r, 64, bn / 2);
  ok = ok && make_bf16_tmap(&tmY, Y, s.d_out, s.T, s.d_out, 64, kBlockM);
  if (!ok) return LORA_ERR_CUDA;
  GemmParams p{};
  p.out = static_cast<__nv_bfloat16*>(Y);
  p.ld_out = static_cast<int>(s.d_out);
  p.M = static_cast<int>(s.T);
  p.N = static_cast<int>(s.d_out);
  p.K = static_cast<int>(s.d_in);
  p.r_pad = r;
  p.block_n = bn;
  p.tiles_m = ceil_div(s.T, kPairBlockM);
  p.tiles_n = ceil_div(s.d_out, bn);
  p.num_tiles = p.tiles_m * p.tiles_n;
  p.kblocks = ceil_div(s.d_in, kBlockK);
  p.group_m = pl->cfg.group_m;
  p.stages = 6;
  p.tail_delay = pl->cfg.tail_delay;
  p.scale = scale;
  p.kb_per_split = p.kblocks;
  p.split_k = 1;
  p.ld_rt = pl->ws.ld_t;
  p.status = pl->d_status;
  p.wait_limit = pl->wait_limit;
  p.tail_parts = 1;
  p.n_groups = pl->n_groups;
  for (int g = 0; g < pl->n_groups; ++g) p.group_end[g] = static_cast<int>(pl->group_off[g + 1]);
  const int ctas = 2 * (p.num_tiles < pairs ? p.num_tiles : pairs);
  if (launch_gemm_pair_fwd_ext(tmX, tmW, tmPt, tmB, tmY, p, ctas, st) != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  return LORA_OK;
}

// dX GEMM over the concatenated contraction (all groups' dY columns), plus one rank-r k-block per group
int launch_grouped_dx_gemm(lora_plan* pl, const void* dY, const void* W, const void* A, float scale, void* dX, cudaStream_t st) {
  const lora_shape_t& s = pl->shape;
  const int pairs = pl->num_sms / 2, r = static_cast<int>(s.r), R = pl->n_groups * r;
  uint8_t* ws = static_cast<uint8_t*>(pl->workspace);
  const int bn = pick_pair_block_n(s.T, s.d_in, 0, pairs);
  CUtensorMap tmdY, tmW, tmQt, tmA, tmdX;
  bool ok = make_bf16_tmap(&tmdY, dY, s.d_out, s.T, s.d_out, 64, kBlockM);
  ok = ok && make_bf16_tmap(&tmW, W, s.d_in, s.d_out, s.d_in, 64, 64);
  ok = ok && make_bf16_tmap(&tmQt, ws + pl->gws.qt, s.T, R, pl->ws.ld_t, 64, r);
  ok = ok && make_bf16_tmap(&tmA, A, s.d_in, R, s.d_in, 64, r);
  ok = ok && make_bf16_tmap(&tmdX, dX, s.d_in, s.T, s.d_in, 64, kBlockM);
  if (!ok) return LORA_ERR_CUDA;
  GemmParams p{};
  p.out = static_cast<__nv_bfloat16*>(dX);
  p.ld_out = static_cast<int>(s.d_in);
  p.M = static_cast<int>(s.T);
  p.N = static_cast<int>(s.d_in);
  p.K = static_cast<int>(s.d_out);
  p.r_pad = r;
  p.block_n = bn;
  p.tiles_m = ceil_div(s.T, kPairBlockM);
  p.tiles_n = ceil_div(s.d_in, bn);
  p.num_tiles = p.tiles_m * p.tiles_n;
  p.kblocks = ceil_div(s.d_out, kBlockK);
  p.group_m = pl->cfg.group_m;
  p.stages = 6;
  p.tail_delay = pl->cfg.tail_delay;
  p.scale = scale;
  p.kb_per_split = p.kblocks;
  p.split_k = 1;
  p.ld_rt = pl->ws.ld_t;
  p.status = pl->d_status;
  p.wait_limit = pl->wait_limit;
  p.tail_parts = pl->n_groups;
  const int ctas = 2 * (p.num_tiles < pairs ? p.num_tiles : pairs);
  if (launch_gemm_pair_dx(tmdY, tmW, tmQt, tmA, tmdX, p, ctas, st) != cudaSuccess) return LORA_ERR_CUDA;
  g_launches.fetch_add(1);
  return LORA_OK;
}

int check_group_shape(const lora_group_shape_t* g) {
  if (g == nullptr) return LORA_ERR_INVALID_ARG;
  if (g->T <= 0 || g->d_in <= 0 || g->r <= 0 || g->n_groups < 2 || g->n_groups > 4) return LORA_ERR_INVALID_ARG;
  if (g->T <= kBlockM || g->T > (1ll << 30) || g->d_in > (1ll << 24) || g->d_in % 8 != 0) return LORA_ERR_UNSUPPORTED_SHAPE;
  if (g->r % 16 != 0 || g->r > 64) return LORA_ERR_UNSUPPORTED_SHAPE;        // a group's rows are whole 16-row MMA k-steps
  const int n_jobs_sides = g->n_groups + ceil_div(g->n_groups * g->r, kGroupRowsPerJob);
  if (n_jobs_sides > kGradMaxJobs) return LORA_ERR_UNSUPPORTED_SHAPE;
  long long total = 0;
  for (int i = 0; i < g->n_groups; ++i) {
    if (g->d_out[i] <= 0) return LORA_ERR_INVALID_ARG;
    if (g->d_out[i] % 256 != 0) return LORA_ERR_UNSUPPORTED_SHAPE;            // output tiles must not straddle two groups
    total += g->d_out[i];
  }
  if (total > (1ll << 24)) return LORA_ERR_UNSUPPORTED_SHAPE;
  return LORA_OK;
}

}  // namespace

extern "C" {

int lora_plan_create_grouped(const lora_group_shape_t* gshape, int device, lora_plan_t** out) {
  if (out == nullptr) return LORA_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = check_group_shape(gshape);
  if (rc != LORA_OK) return rc;
  lora_shape_t flat;
  flat.T = gshape->T;
  flat.d_in = gshape->d_in;
  flat.r = gshape->r;
  flat.d_out = 0;
  for (int i = 0; i < gshape->n_groups; ++i) flat.d_out += gshape->d_out[i];
  lora_plan_t* pl = nullptr;
  rc = lora_plan_create(&flat, device, &pl);
  if (rc != LORA_OK) return rc;
  if (pl->num_sms < 2 * kGradMaxJobs) {
    lora_plan_destroy(pl);
    return LORA_ERR_NO_DEVICE;
  }
  pl->n_groups = gshape->n_groups;
  pl->group_off[0] = 0;
  for (int i = 0; i < gshape->n_groups; ++i) pl->group_off[i + 1] = pl->group_off[i] + gshape->d_out[i];
  // workspace: the stacked products of all groups, one partial-sum region and one counter range per streaming job
  const size_t R = static_cast<size_t>(gshape->n_groups) * gshape->r;
  size_t off = 0;
  pl->gws.qt = off;     off += align_up(R * pl->ws.ld_t * 2, kAlign);
  pl->gws.pt = off;     off += align_up(R * pl->ws.ld_t * 2, kAlign);
  pl->gws.part_stride = align_up(static_cast<size_t>(kSideMaxChunks) * kGroupRowsPerJob * pl->ws.ld_t * 4, kAlign);
  pl->gws.part = off;   off += kGradMaxJobs * pl->gws.part_stride;
  pl->gws.count = off;  off += align_up(static_cast<size_t>(kGradMaxJobs) * pl->ws.n_slabs * sizeof(int), kAlign);
  pl->gws.total = off;
  pl->ws.total = off;                                     // what lora_plan_workspace_bytes / lora_plan_set_workspace go by
  *out = pl;
  return LORA_OK;
}

int lora_linear_fwd_grouped(lora_plan_t* plan, const void* X, const void* W_cat, const void* A_cat, const void* B_cat, float scale,
                            void* Y_cat, void* stream) {
  if (plan == nullptr || plan->n_groups < 2) return LORA_ERR_INVALID_ARG;
  if (!X || !W_cat || !A_cat || !B_cat || !Y_cat) return LORA_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(W_cat) || !aligned16(A_cat) || !aligned16(B_cat) || !aligned16(Y_cat)) return LORA_ERR_MISALIGNED;
  if (plan->workspace == nullptr || plan->workspace_bytes < plan->ws.total) return LORA_ERR_WORKSPACE;
  DeviceGuard guard(plan->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = launch_grouped_sides(plan, nullptr, nullptr, X, A_cat, scale, false, st);      // Pt_all = s (X A_cat^T)^T
  if (rc == LORA_OK) rc = launch_grouped_fwd_gemm(plan, X, W_cat, B_cat, scale, Y_cat, st);
  return rc;
}

int lora_linear_bwd_grouped(lora_plan_t* plan, const void* dY_cat, const void* X, const void* W_cat, const void* A_cat,
                            const void* B_cat, float scale, void* dX, void* dA_cat, void* dB_cat, void* stream) {
  if (plan == nullptr || plan->n_groups < 2) return LORA_ERR_INVALID_ARG;
  if (!dY_cat || !X || !W_cat || !A_cat || !B_cat || !dX || !dA_cat || !dB_cat) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dY_cat) || !aligned16(X) || !aligned16(W_cat) || !aligned16(A_cat) || !aligned16(B_cat) || !aligned16(dX) ||
      !aligned16(dA_cat) || !aligned16(dB_cat))
    return LORA_ERR_MISALIGNED;
  if (plan->workspace == nullptr || plan->workspace_bytes < plan->ws.total) return LORA_ERR_WORKSPACE;
  DeviceGuard guard(plan->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = launch_grouped_sides(plan, dY_cat, B_cat, X, A_cat, scale, true, st);          // Qt_all and Pt_all, one launch
  if (rc == LORA_OK) rc = launch_grouped_dx_gemm(plan, dY_cat, W_cat, A_cat, scale, dX, st);
  if (rc == LORA_OK) rc = launch_grouped_grads(plan, dY_cat, X, dA_cat, dB_cat, st);
  return rc;
}

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
  pl->d_status = nullptr;
  if (gemm_configure() != cudaSuccess || gemm_pair_configure() != cudaSuccess || grad_configure() != cudaSuccess || encode_fn() == nullptr) {
    cudaGetLastError();
    delete pl;
    return LORA_ERR_CUDA;
  }
  device_caps(device, pl->num_sms, pl->caps);
  rc = select_config(shape, pl->num_sms, &pl->cfg, pl->caps);
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
  pl->counters_clean = false;
  pl->n_groups = 0;
  if (const char* f = std::getenv("LORA_LOG")) {          // LORA_LOG=1: one line per plan with what the selector chose
    if (std::atoi(f) != 0) {
      char line[1024];
      lora_plan_describe(pl, line, sizeof(line));
      std::fprintf(stderr, "[lora_linear] plan %p: %s\n", static_cast<void*>(pl), line);
    }
  }
  if (cudaMalloc(&pl->d_status, 256) != cudaSuccess || cudaMemset(pl->d_status, 0, 256) != cudaSuccess) {
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
  delete plan;
  return LORA_OK;
}

int lora_plan_workspace_bytes(const lora_plan_t* plan, size_t* fwd_bytes, size_t* bwd_bytes) {
  if (plan == nullptr) return LORA_ERR_INVALID_ARG;
  if (fwd_bytes) *fwd_bytes = (plan->n_groups != 0 || (plan->cfg.cta_group == 2 && plan->cfg.fwd_ext)) ? plan->ws.total : 0;
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
  plan->counters_clean = false;
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
  g.tmem_cols = grad_tmem_cols(g.feat_chunk, r_pad, true, false);
  g.do_out = 1;
  g.scale = 1.f;
  g.out = static_cast<float*>(out);
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
                "split_k=%d/%d r_pad=%d ctas fwd=%d dx=%d tail_delay=%d | grad chunk=%d/%d stages=%d/%d dA grid=%dx%d%s dB grid=%dx%d "
                "(feature chunks x cluster of token chunks) | bwd workspace=%zu B",
                (long long)plan->shape.T, (long long)plan->shape.d_in, (long long)plan->shape.d_out,
                (long long)plan->shape.r, plan->num_sms, c.cta_group, c.block_m, c.fwd_block_n, c.block_m, c.dx_block_n,
                c.stages, c.dx_stages, c.group_m, c.split_k, c.dx_split_k,
                c.r_pad, c.fwd_ctas, c.dx_ctas, c.tail_delay, c.grad_feat_chunk, c.db_feat_chunk, c.grad_stages, c.db_stages,
                c.da_feat_chunks,
                c.da_token_chunks, c.da_with_p ? " +XA^T" : " (XA^T in its own pass)", c.db_feat_chunks, c.db_token_chunks, plan->ws.total);
  return LORA_OK;
}

int lora_linear_fwd(lora_plan_t* plan, const void* X, const void* W, const void* A, const void* B, float scale,
                    void* Y, void* stream) {
  if (plan == nullptr || plan->n_groups != 0) return LORA_ERR_INVALID_ARG;
  if (plan->shape.T == 0) return LORA_OK;
  if (!X || !W || !A || !B || !Y) return LORA_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(W) || !aligned16(A) || !aligned16(B) || !aligned16(Y)) return LORA_ERR_MISALIGNED;
  DeviceGuard guard(plan->device);
  return launch_fwd(plan, X, W, A, B, scale, Y, static_cast<cudaStream_t>(stream));
}

int lora_linear_bwd(lora_plan_t* plan, const void* dY, const void* X, const void* W, const void* A, const void* B,
                    float scale, void* dX, void* dA, void* dB, void* stream) {
  if (plan == nullptr || plan->n_groups != 0) return LORA_ERR_INVALID_ARG;
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
  int rc = LORA_OK;
  bool p_ready = false;
  if (plan->cfg.bwd_merged && plan->cfg.cta_group == 2) {
    rc = launch_side_pair(plan, dY, B, X, A, scale, st);        // s (dY B)^T and s (X A^T)^T in one launch
    plan->q_ready = p_ready = true;
  }
  if (rc == LORA_OK) rc = launch_dx(plan, dY, W, A, B, scale, dX, st);
  plan->q_ready = false;
  if (rc == LORA_OK) rc = launch_adapter_grads(plan, dY, X, A, scale, dA, dB, p_ready, st);
  return rc;
}

int lora_linear_bwd_sides(lora_plan_t* plan, const void* dY, const void* X, const void* A, const void* B, float scale,
                          void* stream) {
  if (plan == nullptr) return LORA_ERR_INVALID_ARG;
  if (plan->shape.T == 0) return LORA_OK;
  if (!dY || !X || !A || !B) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(X) || !aligned16(A) || !aligned16(B)) return LORA_ERR_MISALIGNED;
  if (plan->workspace == nullptr || plan->workspace_bytes < plan->ws.total) return LORA_ERR_WORKSPACE;
  DeviceGuard guard(plan->device);
  const int rc = launch_side_pair(plan, dY, B, X, A, scale, static_cast<cudaStream_t>(stream));
  if (rc == LORA_OK) plan->q_staged = plan->cfg.cta_group == 2;    // the single-CTA dX kernel computes dY B itself
  return rc;
}

int lora_linear_bwd_grads(lora_plan_t* plan, const void* dY, const void* X, const void* A, float scale, void* dA, void* dB,
                          void* stream) {
  if (plan == nullptr || !dA || !dB) return LORA_ERR_INVALID_ARG;
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
  if (!dY || !X || !A) return LORA_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(X) || !aligned16(A)) return LORA_ERR_MISALIGNED;
  if (plan->workspace == nullptr || plan->workspace_bytes < plan->ws.total) return LORA_ERR_WORKSPACE;
  return launch_grad_pair(plan, X, dY, A, scale, dA, dB, st);
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
  return launch_da_stage(plan, X, A, scale, dA, static_cast<cudaStream_t>(stream));
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
  if (w_scratch != nullptr && nf4_banded(plan)) {
    const int rcb = check_nf4_banded(plan);
    if (rcb != LORA_OK) return rcb;
    return launch_fwd_nf4_banded(plan, X, W_codes, W_absmax, A, B, scale, Y, w_scratch, st);
  }
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
  if (w_scratch != nullptr && nf4_banded(plan)) {
    int rcb = check_nf4_banded(plan);
    if (rcb != LORA_OK) return rcb;
    bool p_ready = false;
    if (plan->cfg.bwd_merged) {
      rcb = launch_side_pair(plan, dY, B, X, A, scale, st);
      plan->q_ready = p_ready = true;
    }
    if (rcb == LORA_OK) rcb = launch_dx_nf4_banded(plan, dY, W_codes, W_absmax, A, B, scale, dX, w_scratch, st);
    plan->q_ready = false;
    if (rcb == LORA_OK) rcb = launch_adapter_grads(plan, dY, X, A, scale, dA, dB, p_ready, st);
    return rcb;
  }
  if (w_scratch != nullptr) {
    if (plan->workspace == nullptr || plan->workspace_bytes < plan->ws.total) return LORA_ERR_WORKSPACE;
    if (launch_nf4_dequantize(static_cast<const uint8_t*>(W_codes), static_cast<const float*>(W_absmax), plan->shape.d_out,
                              plan->shape.d_in, static_cast<__nv_bfloat16*>(w_scratch), plan->num_sms, st) != cudaSuccess)
      return LORA_ERR_CUDA;
    g_launches.fetch_add(1);
    int rc2 = LORA_OK;
    bool p_ready = false;
    if (plan->cfg.bwd_merged && plan->cfg.cta_group == 2) {
      rc2 = launch_side_pair(plan, dY, B, X, A, scale, st);
      plan->q_ready = p_ready = true;
    }
    if (rc2 == LORA_OK) rc2 = launch_dx(plan, dY, w_scratch, A, B, scale, dX, st);
    plan->q_ready = false;
    if (rc2 == LORA_OK) rc2 = launch_adapter_grads(plan, dY, X, A, scale, dA, dB, p_ready, st);
    return rc2;
  }
  int rc = check_nf4(plan);
  if (rc != LORA_OK) return rc;
  bool p_ready = false;
  if (plan->cfg.bwd_merged) {
    rc = launch_side_pair(plan, dY, B, X, A, scale, st);
    plan->q_ready = p_ready = true;
  }
  if (rc == LORA_OK) rc = launch_dx_nf4(plan, dY, W_codes, W_absmax, A, B, scale, dX, st);
  plan->q_ready = false;
  if (rc == LORA_OK) rc = launch_adapter_grads(plan, dY, X, A, scale, dA, dB, p_ready, st);
  return rc;
}

int lora_plan_nf4_scratch_bytes(const lora_plan_t* plan, size_t* min_bytes, size_t* full_bytes) {
  if (plan == nullptr || plan->n_groups != 0) return LORA_ERR_INVALID_ARG;
  if (min_bytes) *min_bytes = nf4_min_bytes(plan);
  if (full_bytes) *full_bytes = nf4_full_bytes(plan);
  return LORA_OK;
}

int lora_plan_set_nf4_scratch_bytes(lora_plan_t* plan, size_t bytes) {
  if (plan == nullptr || plan->n_groups != 0) return LORA_ERR_INVALID_ARG;
  if (bytes != 0 && bytes < nf4_full_bytes(plan)) {
    const lora_kernel_config_t& c = plan->cfg;
    if (c.cta_group != 2 || c.split_k != 1 || c.dx_split_k != 1) return LORA_ERR_UNSUPPORTED_SHAPE;
    if (bytes < nf4_min_bytes(plan)) return LORA_ERR_WORKSPACE;
  }
  plan->nf4_scratch_bytes = bytes;
  return LORA_OK;
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
  plan->counters_clean = false;      // an abandoned launch may have left arrival counters behind
  return LORA_OK;
}

int lora_plan_last_gemm_clock(lora_plan_t* plan, void* stream, double* sm_mhz, double* busy_us) {
  if (plan == nullptr || sm_mhz == nullptr || busy_us == nullptr) return LORA_ERR_INVALID_ARG;
  DeviceGuard guard(plan->device);
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return LORA_ERR_CUDA;
  unsigned long long rec[4] = {0, 0, 0, 0};
  if (cudaMemcpy(rec, reinterpret_cast<unsigned char*>(plan->d_status) + 64, sizeof(rec), cudaMemcpyDeviceToHost) != cudaSuccess)
    return LORA_ERR_CUDA;
  *sm_mhz = 0.0;
  *busy_us = 0.0;
  if (rec[1] > rec[0] && rec[3] > rec[2]) {
    const double ns = static_cast<double>(rec[1] - rec[0]);
    *busy_us = ns * 1e-3;
    *sm_mhz = static_cast<double>(rec[3] - rec[2]) / ns * 1e3;     // ticks per nanosecond -> MHz
  }
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
