"""Host-side checks that need no GPU: the library loads, exports what include/kvp.h declares,
its layer-map helpers agree with Table 1 of the paper, and kvp_create validates its input."""
import os
import re

import pytest

import workloads as wl
from conftest import ROOT, read_layer_map_golden


@pytest.fixture(scope="module")
def kvp():
    import __graft_entry__ as ge
    ge.build()
    import paper_2410_08391_b200 as k
    return k


def test_library_exports_every_declared_symbol(kvp):
    hdr = open(os.path.join(ROOT, "include", "kvp.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(kvp_[a-z_0-9]+)\s*\(", hdr))
    assert {"kvp_create", "kvp_load_weights", "kvp_prefill_predict", "kvp_decode_step"} <= declared
    L = kvp.lib()
    for name in declared:
        assert hasattr(L, name), f"{name} declared in kvp.h but not exported"
    assert declared == set(kvp.binding.EXPORTS)


@pytest.mark.parametrize("row", read_layer_map_golden(), ids=lambda r: r["name"])
def test_layer_map_helpers_match_table_1(kvp, row):
    if row["kind"] == "C":
        got = kvp.kvp_layer_map_canonical(row["n_base"], row["n_aux"])
    else:
        got = kvp.kvp_layer_map_pruned(row["n_base"], row["retained"])
    assert got == row["map"]


def test_layer_map_uniform(kvp):
    assert kvp.kvp_layer_map_uniform(4, 2) == [0, 0, 1, 1]
    assert kvp.kvp_layer_map_uniform(28, 16) == list(wl.pair("c2").layer_map)
    with pytest.raises(kvp.KvpError):
        kvp.kvp_layer_map_canonical(4, 8)
    with pytest.raises(kvp.KvpError):
        kvp.kvp_layer_map_pruned(8, [1, 2])


def test_create_validates(kvp):
    p = wl.pair("c1")
    h = kvp.kvp_create(p.aux, p.base, p.layer_map, "f32")
    assert kvp.kvp_packed_weight_bytes(h) > 0
    assert kvp.kvp_workspace_bytes(h, 1, 64) > 0
    assert kvp.kvp_cache_layout(h, 0) == 4 * 64 * 16 * 4
    with pytest.raises(kvp.KvpError) as e:
        kvp.kvp_cache_layout(h, 99)
    assert e.value.status == -1
    kvp.kvp_destroy(h)
    for bad_map in [(0, 0, 1, 2), (0, 1, 0, 1), (-1, 0, 1, 1)]:
        with pytest.raises(kvp.KvpError) as e:
            kvp.kvp_create(p.aux, p.base, bad_map, "f32")
        assert e.value.status == -1
    other = wl.uniform_model(4, 128, 8, 4, 16, 344, 513)      # vocabulary differs from the aux model's
    with pytest.raises(kvp.KvpError) as e:
        kvp.kvp_create(p.aux, other, p.layer_map, "f32")
    assert e.value.status == -2
    odd = wl.uniform_model(2, 64, 4, 3, 16, 172, 512)          # 4 q heads over 3 kv heads
    with pytest.raises(kvp.KvpError) as e:
        kvp.kvp_create(odd, p.base, p.layer_map, "f32")
    assert e.value.status == -2
    with pytest.raises(kvp.KvpError) as e:
        kvp.kvp_create(p.aux, p.base, p.layer_map, "f32", page_tokens=16)
    assert e.value.status == -1


def test_all_configs_plan(kvp):
    for name in ("c1", "c2", "c3", "c4", "c5"):
        p = wl.pair(name)
        h = kvp.kvp_create(p.aux, p.base, p.layer_map, p.dtype)
        pr_total = {"c1": 64, "c2": 1024, "c3": 8 * 4096, "c4": 65536, "c5": 65536}[name]
        nb = {"c1": 1, "c2": 1, "c3": 8, "c4": 32, "c5": 4}[name]
        assert kvp.kvp_workspace_bytes(h, nb, pr_total) < 40e9
        es = 2 if p.dtype == "bf16" else 4
        n_params = sum(int(__import__("numpy").prod(s)) for s in wl.weight_shapes(p).values())
        assert kvp.kvp_packed_weight_bytes(h) >= 0.9 * n_params * es * (1 if name != "c4" else 0.5)
        kvp.kvp_destroy(h)
