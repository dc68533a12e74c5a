"""CPU-only checks of the C-ABI boundary: the library builds for sm_100a, loads, and exports
every function declared in include/selectinfer.h and include/selectinfer_debug.h.  No compute call is made."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for header in ("selectinfer.h", "selectinfer_debug.h"):
        text = open(os.path.join(ROOT, "include", header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names.update(re.findall(r"\b(si_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2607_18081_b200 import build
    path = build.build()
    import torch  # noqa: F401  makes libcudart resolvable
    lib = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), f"{n} declared in selectinfer.h but not exported"
    for required in ("si_load_neurons", "si_select", "si_ffn_forward", "si_layer_forward"):
        assert required in names


def test_binding_names_match_header_and_host_side_errors():
    from paper_2607_18081_b200 import api
    names = _declared()
    for n in names:
        assert n in api.EXPORTS or hasattr(api, n), n
    for n in api.EXPORTS:
        assert n in names, f"binding lists {n} which the header does not declare"
    assert api.strerror(0) == "ok" and "range" in api.strerror(api.SI_ERR_OUT_OF_RANGE)
    assert "sm_100a" in api.build_info()
    # host-checkable argument errors need no GPU: bad shapes are refused before any CUDA call
    out = ctypes.c_size_t(0)
    n_loaded = (ctypes.c_int * 1)(10)
    assert api.lib().si_store_bytes(1, 100, 64, n_loaded, api.SI_BF16, ctypes.byref(out)) == api.SI_ERR_INVALID_ARG
    assert api.lib().si_store_bytes(1, 128, 64, n_loaded, 7, ctypes.byref(out)) == api.SI_ERR_INVALID_ARG
    assert api.lib().si_store_bytes(1, 128, 64, n_loaded, api.SI_BF16, ctypes.byref(out)) == api.SI_OK
    assert out.value >= 10 * 3 * 128 * 2 + 10 * 4 + 64 * 4
    n_loaded[0] = 65
    assert api.lib().si_store_bytes(1, 128, 64, n_loaded, api.SI_BF16, ctypes.byref(out)) == api.SI_ERR_INVALID_ARG
    assert api.lib().si_select(None, 4, 0, 1, 0.0, 0, None, 4, None, None, 0, None) == api.SI_ERR_INVALID_ARG


def test_store_bytes_is_eq2_accounting():
    """Bytes kept for the records = 3*d*e*n_loaded; bytes not stored = Eq. 2 with r_layer = 1."""
    from paper_2607_18081_b200 import api
    from oracle import selectinfer_oracle as so
    L, d, F = 4, 4096, 11008
    n_ld = so.count_from_pct(70, F)
    total = api.si_store_bytes(L, d, F, [n_ld] * L, "bf16")
    records = L * n_ld * 3 * d * 2
    maps = total - records
    assert 0 <= maps <= L * (n_ld * 4 + F * 4 + 3 * 256)
    full = L * 3 * d * F * 2
    saving = so.memory_saving(L * 3 * d * F, n_ld / F, 1.0, 2)
    assert abs((full - records) - saving) < 1e-6 * full


def test_layer_range_matches_the_papers_layer_counts():
    """Host-only entry point: Table 1's layer policy gives the layer counts of the paper's evaluation."""
    from oracle import selectinfer_oracle as so
    from paper_2607_18081_b200 import api
    from tests.helpers import paper_values
    pv = paper_values()
    first, last = int(pv["table1_first_layer"]), int(pv["table1_last_layer"])
    for n_layers in (int(pv["llama32_1b_layers"]), int(pv["llama32_3b_layers"]), 32):
        lo, hi = api.si_layer_range(n_layers, first, last)
        assert list(range(lo, hi)) == so.layer_range(n_layers, first, last)
    lo, hi = api.si_layer_range(int(pv["llama32_1b_layers"]), first, last)
    assert hi - lo == pv["llama32_1b_selective_layers"]
    import pytest
    with pytest.raises(api.SelectInferError):
        api.si_layer_range(6, 5, -2)


def test_shard_entry_points_host_side():
    """Neuron shards: the share sizes and the argument checks need no GPU."""
    from paper_2607_18081_b200 import api
    for n, world in ((10, 3), (7705, 8), (5, 8), (0, 2), (1, 1)):
        counts = [api.si_shard_count(n, r, world) for r in range(world)]
        assert sum(counts) == n and max(counts) - min(counts) <= 1
        assert counts == [len(range(r, n, world)) for r in range(world)]
    lib, null = api.lib(), ctypes.c_void_p(0)
    out = ctypes.c_int(0)
    assert lib.si_shard_count(10, 3, 3, ctypes.byref(out)) == api.SI_ERR_INVALID_ARG       # rank outside the world
    assert lib.si_shard_count(10, 0, 0, ctypes.byref(out)) == api.SI_ERR_INVALID_ARG
    assert lib.si_shard_count(-1, 0, 2, ctypes.byref(out)) == api.SI_ERR_INVALID_ARG
    # null outputs, a rank outside the world, a workspace that is too small: refused before any launch
    buf = ctypes.c_void_p(0x1000)
    assert lib.si_shard_lists(buf, null, 4, 2, 0, 2, null, buf, buf, 4096, null, null) == api.SI_ERR_INVALID_ARG
    assert lib.si_shard_lists(buf, null, 4, 2, 2, 2, buf, buf, buf, 4096, null, null) == api.SI_ERR_INVALID_ARG
    assert lib.si_shard_lists(buf, null, 4, 2, 0, 2, buf, buf, buf, 16, null, null) == api.SI_ERR_NOMEM
    assert lib.si_shard_reduce(null, 2, null, api.SI_BF16, 1, 64, buf, api.SI_F32, 0, null) == api.SI_ERR_INVALID_ARG
    assert lib.si_shard_reduce(buf, 0, null, api.SI_BF16, 1, 64, buf, api.SI_F32, 0, null) == api.SI_ERR_INVALID_ARG
    assert lib.si_shard_reduce(buf, 2, null, api.SI_BF16, 1, 64, buf, api.SI_F32, api.SI_FLAG_RESIDUAL, null) == \
        api.SI_ERR_INVALID_ARG                                                              # residual without x
    assert lib.si_shard_reduce(buf, 2, null, api.SI_F32, 1, 64, buf, api.SI_F32, 0, null) == api.SI_ERR_INVALID_ARG


def test_kernel_shapes_of_calls_with_many_tokens():
    """Host logic: which tile shapes a call with more than 128 tokens gets (gate/up: neurons per sub-tile, sub-tiles per
    tile; down: columns per pair tile, K split), on a device of 148 SMs = 74 SM pairs.  The choice minimises waves of
    pair tiles x the time of a tile's chunk."""
    from paper_2607_18081_b200 import api
    # config 4: 512 tokens, union of 3082 slots (room for 3200), d_model 4096.  Tiles of 128 neurons would be 25 x 2 = 50
    # pairs, tiles of 96 are 34 x 2 = 68: still one wave, a quarter less work per pair.  Down: 16 x 2 tiles of 256
    # columns would use 64 SMs, so two pairs share a tile, half of K each: 32 x 4 = 128 CTAs.
    p = api.si_debug_pair_plan(4096, 3200, 512, 148)
    assert (p["gateup_w"], p["gateup_sub"], p["gateup_pairs"]) == (96, 1, 68)
    assert (p["down_n"], p["down_ksplit"], p["down_ctas"]) == (256, 2, 128)
    # all 7705 loaded neurons (room for 7808): 122 tiles of 128 would be two waves; 35 x 2 = 70 tiles of 2 x 112 are one
    p = api.si_debug_pair_plan(4096, 7808, 512, 148)
    assert (p["gateup_w"], p["gateup_sub"], p["gateup_pairs"]) == (112, 2, 70)
    assert (p["down_n"], p["down_ksplit"]) == (256, 2)
    # a union of 4608 slots is exactly 36 x 2 = 72 tiles of 128: one full wave, nothing to gain from narrower tiles
    p = api.si_debug_pair_plan(4096, 4608, 512, 148)
    assert (p["gateup_w"], p["gateup_sub"], p["gateup_pairs"]) == (128, 1, 72)
    # 2048 tokens: 8 token tiles x 16 column tiles of 256 fill the machine without a K split
    p = api.si_debug_pair_plan(4096, 3200, 2048, 148)
    assert (p["down_n"], p["down_ksplit"], p["down_ctas"]) == (256, 1, 256)
    # a short K (room for 1024 slots: 16 chunks) does not pay for the exchange of a K split: tiles of 128 columns
    p = api.si_debug_pair_plan(4096, 1024, 512, 148)
    assert (p["down_n"], p["down_ksplit"], p["down_ctas"]) == (128, 1, 128)
    # a hidden size that is no multiple of 256 (640) has 128-column tiles only
    p = api.si_debug_pair_plan(640, 768, 200, 148)
    assert (p["down_n"], p["down_ksplit"], p["down_ctas"]) == (128, 1, 10)
    for bad in ((4096, 3200, 128, 148), (4000, 3200, 512, 148), (4096, 3000, 512, 148), (4096, 0, 512, 148)):
        with pytest.raises(api.SelectInferError) as e:
            api.si_debug_pair_plan(*bad)
        assert e.value.status == api.SI_ERR_INVALID_ARG
