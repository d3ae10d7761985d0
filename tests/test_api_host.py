"""Host-side checks that need no GPU: the library loads, exports what include/lora_linear.h
declares, and the selector / workspace / argument checks behave."""
import ctypes
import os
import re

import pytest

from paper_2503_22673_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "lora_linear.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lora_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    names = _declared_symbols()
    assert "lora_linear_fwd" in names and "lora_linear_bwd" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_strerror_and_launch_count():
    assert binding.strerror(0) == "ok"
    assert "shape" in binding.strerror(binding.LORA_ERR_UNSUPPORTED_SHAPE)
    assert binding.strerror(-12345) == "unknown status"
    assert binding.launch_count() >= 0


@pytest.mark.parametrize("shape", [(8192, 4096, 4096, 16), (16384, 4096, 14336, 16), (16384, 14336, 4096, 64),
                                   (256, 512, 512, 8), (32768, 4096, 1024, 16), (1, 8, 8, 8), (300, 520, 200, 24)])
def test_selector_invariants(shape):
    T, d_in, d_out, r = shape
    c = binding.select_config(T, d_in, d_out, r, 148)
    assert c["block_k"] == 64
    assert c["r_pad"] % 16 == 0 and r <= c["r_pad"] < r + 16
    assert c["cta_group"] == (2 if T > 128 else 1)
    if c["cta_group"] == 2:
        assert c["block_m"] == 256
        dr = d_out * c["r_pad"]
        assert c["fwd_ext"] == (1 if dr >= 100000 or (dr >= 65536 and T >= 4096) else 0)
        # fused forward: tile + adapter columns share one MMA; K-extended forward: no adapter columns
        assert c["fwd_block_n"] % 16 == 0 and c["fwd_block_n"] + (0 if c["fwd_ext"] else c["r_pad"]) <= 256
        assert c["dx_block_n"] % 16 == 0 and c["dx_block_n"] <= 256                  # K-extended GEMM: no adapter columns
        units = 74                                                  # CTA pairs
        per = 2
        assert c["stages"] * 32768 + 2 * 16384 + 2048 <= 232448     # forward ring + staging fit 227 KiB
        assert c["dx_stages"] * 32768 + 2 * 16384 + 2048 <= 232448
        assert c["q_feat_chunk"] % 128 == 0 and c["q_feat_chunks"] == -(-d_out // c["q_feat_chunk"])
        assert 1 <= c["q_feat_chunks"] * c["q_token_chunks"] <= 148 and c["q_token_chunks"] <= -(-T // 128)
        assert c["q_stages"] * (32768 + 16384) + 4 * c["r_pad"] * 128 + 2048 <= 232448
    else:
        assert c["block_m"] == 128
        for bn in (c["fwd_block_n"], c["dx_block_n"]):
            assert bn in (64, 128, 192) and bn + c["r_pad"] <= 256
        units, per = 148, 1
        assert c["stages"] * (128 * 128 + 256 * 128) + 2 * 16384 + 2048 <= 232448
    m_tiles = -(-T // c["block_m"])
    assert per <= c["fwd_ctas"] <= per * min(units, m_tiles * -(-d_out // c["fwd_block_n"]))
    assert per <= c["dx_ctas"] <= per * min(units, m_tiles * -(-d_in // c["dx_block_n"]))
    assert c["fwd_ctas"] % per == 0 and c["dx_ctas"] % per == 0
    assert 1 <= c["split_k"] <= 8 and 1 <= c["dx_split_k"] <= 8
    if T >= 1024:
        assert c["split_k"] == 1 and c["dx_split_k"] == 1          # the benchmark shapes fill the GPU without it
    n_slabs = -(-T // 128)
    assert c["da_with_p"] == (1 if c["r_pad"] <= 32 else 0)       # large ranks recompute X A^T in their own pass over X
    grids = ((c["grad_feat_chunk"], c["da_feat_chunks"], c["da_token_chunks"], c["grad_stages"], c["da_with_p"], 0, d_in),
             (c["db_feat_chunk"], c["db_feat_chunks"], c["db_token_chunks"], c["db_stages"], 0, 0, d_out),
             (c["dan_feat_chunk"], c["dan_feat_chunks"], c["dan_token_chunks"], c["db_stages"], 0, 0, d_in),
             (c["dbq_feat_chunk"], c["dbq_feat_chunks"], c["dbq_token_chunks"], 4, 1, 1, d_out))
    for fc, nf, nt, st, with_p, side_mn, C in grids:
        assert fc % 128 == 0 and (fc // 128) * c["r_pad"] + with_p * 4 * c["r_pad"] <= 512   # TMEM: sums + side buffers
        assert nf == -(-C // fc)
        assert 1 <= nt <= 16 and nt <= n_slabs                     # the token chunks of a feature chunk are ONE cluster
        assert nf * nt <= 148                                      # resident at once
        assert 2 <= st <= 6
        side = (8192 if side_mn else c["r_pad"] * 128) * 2 * with_p
        assert st * (32768 + side) + 4 * c["r_pad"] * 128 + 2048 <= 232448


def test_selector_band_height_follows_the_weight_size():
    """Rasterisation bands: 2 m-tiles while the weight (at most 48 MiB) stays in L2 whatever the order, 8 for weights of
    L2's own size, which are only reused inside a tall band."""
    assert binding.select_config(8192, 4096, 4096, 16, 148)["group_m"] == 2          # 32 MiB
    assert binding.select_config(32768, 4096, 1024, 16, 148)["group_m"] == 2         # 8 MiB
    assert binding.select_config(16384, 4096, 14336, 16, 148)["group_m"] == 8        # 112 MiB
    assert binding.select_config(16384, 14336, 4096, 64, 148)["group_m"] == 8


def test_selector_grad_grids_of_the_benchmark_shapes():
    """The dA + dB launch of the merged backward: 128-feature blocks of X and dY side by side, each block's token chunks
    one small cluster, so that the grid is as close to the SM count as whole clusters allow."""
    q = binding.select_config(8192, 4096, 4096, 16, 148)
    assert q["bwd_merged"] == 1
    assert (q["pair_feat_chunk"], q["pair_feat_chunks"], q["pair_token_chunks"]) == (128, 64, 2)
    gate = binding.select_config(16384, 4096, 14336, 16, 148)       # 32 + 112 blocks: one CTA each, no sum across CTAs
    assert (gate["pair_feat_chunk"], gate["pair_feat_chunks"], gate["pair_token_chunks"]) == (128, 144, 1)
    down = binding.select_config(16384, 14336, 4096, 64, 148)
    assert (down["pair_feat_chunks"], down["pair_token_chunks"]) == (144, 1) and down["da_with_p"] == 0
    kv = binding.select_config(32768, 4096, 1024, 16, 148)
    assert (kv["pair_feat_chunks"], kv["pair_token_chunks"]) == (40, 3)
    tiny = binding.select_config(256, 512, 512, 8, 148)            # 256 KiB streams: no cluster, nothing summed across CTAs
    assert tiny["da_token_chunks"] == 1 and tiny["db_token_chunks"] == 1 and tiny["pair_token_chunks"] == 1
    for c in (q, gate, down, kv, tiny):
        assert c["pair_feat_chunk"] % 128 == 0 and (c["pair_feat_chunk"] // 128) * c["r_pad"] <= 512
        assert c["pair_feat_chunks"] * c["pair_token_chunks"] <= 148 and 1 <= c["pair_token_chunks"] <= 16


def test_selector_picks_by_grid_size():
    small = binding.select_config(128, 512, 512, 8, 148)          # one 128-row tile: single-CTA kernel, narrow tiles
    big = binding.select_config(16384, 4096, 14336, 16, 148)
    assert small["cta_group"] == 1 and small["fwd_block_n"] == 64 and small["fwd_ctas"] == 8
    assert big["cta_group"] == 2 and big["fwd_ext"] == 1 and big["fwd_block_n"] == 256 and big["fwd_ctas"] == 148
    q = binding.select_config(8192, 4096, 4096, 16, 148)
    assert q["fwd_ext"] == 1 and q["fwd_block_n"] == 256 and q["dx_block_n"] == 256      # pre-pass beats adapter columns
    q_small = binding.select_config(1024, 4096, 4096, 16, 148)                            # few tokens: stay fused
    assert q_small["fwd_ext"] == 0 and q_small["fwd_block_n"] == 240
    kv = binding.select_config(32768, 4096, 1024, 16, 148)        # 1024 columns: 5 x 208 wastes less than 5 x 240
    assert kv["fwd_block_n"] == 208


def test_selector_splits_k_only_for_starved_grids_with_long_contractions():
    skinny = binding.select_config(257, 14336, 264, 64, 148)      # 2 x 2 tiles, 224 k-blocks
    assert skinny["split_k"] == 8 and skinny["fwd_ext"] == 1 and skinny["fwd_ctas"] == 2 * 4 * 8
    assert binding.select_config(256, 4096, 4096, 16, 148)["split_k"] == 1     # 29 tiles: enough parallelism
    assert binding.select_config(300, 2048, 1032, 16, 148)["split_k"] == 1     # 32 k-blocks: too short to pay a reduce
    assert binding.select_config(256, 512, 512, 8, 148)["split_k"] == 1        # workload 0


@pytest.mark.parametrize("bad,code", [((128, 4100, 64, 16), binding.LORA_ERR_UNSUPPORTED_SHAPE),
                                      ((128, 64, 60, 16), binding.LORA_ERR_UNSUPPORTED_SHAPE),
                                      ((128, 64, 64, 12), binding.LORA_ERR_UNSUPPORTED_SHAPE),
                                      ((128, 64, 64, 72), binding.LORA_ERR_UNSUPPORTED_SHAPE),
                                      ((-1, 64, 64, 16), binding.LORA_ERR_INVALID_ARG),
                                      ((128, 0, 64, 16), binding.LORA_ERR_INVALID_ARG)])
def test_selector_rejects_bad_shapes(bad, code):
    with pytest.raises(binding.LoraError) as ei:
        binding.select_config(*bad)
    assert ei.value.code == code
    with pytest.raises(binding.LoraError):
        binding.workspace_bytes(*bad)


def test_workspace_is_small_next_to_the_streams():
    # scratch for Qt, Pt and the fixed-order partial sums; forward needs none
    T, d_in, d_out, r = 8192, 4096, 4096, 16
    ws = binding.workspace_bytes(T, d_in, d_out, r)
    assert 0 < ws < (T * d_in * 2) // 2
    assert binding.workspace_bytes(0, d_in, d_out, r) > 0


def test_null_arguments_are_rejected_without_a_gpu():
    lib = binding.load()
    assert lib.lora_plan_create(None, 0, None) == binding.LORA_ERR_INVALID_ARG
    assert lib.lora_plan_destroy(None) == binding.LORA_ERR_INVALID_ARG
    assert lib.lora_linear_fwd(None, None, None, None, None, 1.0, None, None) == binding.LORA_ERR_INVALID_ARG
    assert lib.lora_linear_bwd(None, None, None, None, None, None, 1.0, None, None, None, None) == \
        binding.LORA_ERR_INVALID_ARG
    assert lib.lora_select_config(None, 148, None) == binding.LORA_ERR_INVALID_ARG
    out = ctypes.c_size_t(0)
    s = binding.LoraShape(128, 64, 64, 16)
    assert lib.lora_step_host_staging_bytes(ctypes.byref(s), ctypes.byref(out)) == 0
    assert out.value >= 2 * 128 * 64 * 2 * 2


def test_plan_creation_fails_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    lib = binding.load()
    h = ctypes.c_void_p(0)
    s = binding.LoraShape(128, 64, 64, 16)
    assert lib.lora_plan_create(ctypes.byref(s), 0, ctypes.byref(h)) == binding.LORA_ERR_NO_DEVICE
    assert not h.value
    with pytest.raises(binding.LoraError):
        binding.LoraLinearPlan(128, 64, 64, 16)
