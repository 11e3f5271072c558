"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, and rejects bad descriptors before touching the device."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2512_17917_b200 import binding, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "kvr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kvr_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = binding.lib()
    names = _declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(binding.EXPORTS)


def test_status_strings():
    assert binding.status_string(0) == "ok"
    assert "unsupported" in binding.status_string(2)
    assert binding.status_string(99) == "unknown status"


def _create(**over):
    kw = dict(r=3, b=8, head_dim=128, n_kv_heads=2, n_q_heads=8, batch=1, n_layers=1, max_context=64,
              kv_dtype=0, index_mix=1, seeds_per_head=0)
    kw.update(over)
    desc = binding.SketchDesc(*[kw[n] for n, _ in binding.SketchDesc._fields_])
    seeds = over.get("_seeds", synth.hash_seeds(1))
    seeds = np.ascontiguousarray(seeds, np.uint32)
    out = ctypes.c_void_p(0)
    st = binding.lib().kvr_sketch_create(ctypes.byref(out), ctypes.byref(desc),
                                         seeds.ctypes.data_as(ctypes.c_void_p), None)
    assert st != 0 and not out.value
    return st


@pytest.mark.parametrize("over,status", [
    (dict(b=0), 1), (dict(batch=0), 1), (dict(max_context=0), 1), (dict(kv_dtype=7), 1),
    (dict(n_q_heads=7), 1), (dict(index_mix=2), 1), (dict(seeds_per_head=2), 1),
    (dict(r=7), 2), (dict(r=2), 2), (dict(head_dim=64), 2), (dict(b=8193), 2), (dict(n_q_heads=6), 2),
    (dict(batch=4096, n_layers=64), 2),
])
def test_create_rejects_bad_descriptors_without_a_device(over, status):
    assert _create(**over) == status


def test_create_rejects_bad_seeds_and_null_pointers():
    bad = synth.hash_seeds(2)
    bad[1, 2] = 2 ** 31 - 1          # seeds must be < p
    assert _create(_seeds=bad) == 1
    L = binding.lib()
    assert L.kvr_sketch_create(None, None, None, None) == 1
    assert L.kvr_compress(None, 0, None, None, None, 1, 1, 1, 0, None, None, None, None) == 1
    assert L.kvr_decode_attention(None, 0, None, None, None, None, 0, 0.0, None, None) == 1
    assert L.kvr_sketch_destroy(None) == 0
    assert L.kvr_sketch_device_bytes(None) == 0


def test_workload_table_matches_the_benchmark_configurations():
    w = synth.WORKLOADS
    assert (w["2k_single_layer"].budget, w["2k_single_layer"].b) == (205, 7)
    assert (w["32k_llama3_8b"].budget, w["32k_llama3_8b"].b, w["32k_llama3_8b"].n_inst) == (8192, 273, 256)
    assert w["32k_llama3_8b_batch16"].n_inst == 4096 and w["32k_llama3_8b_batch16"].dtype == "bf16"
    assert w["8k_qwen3_8b_batch8"].n_inst == 2304
    assert synth.default_sketch_width(819, 3, 0.5) == 14 and synth.default_sketch_width(819, 3, 2.0) == 55


def test_paper_storage_split_matches_the_oracle():
    """Host arithmetic of the C ABI against the oracle's restatement of the paper's split."""
    import pytest
    import paper_2512_17917_b200 as kvr
    from oracle import kvr_oracle as orc
    for N in (1, 7, 100, 2048, 8192, 32768, 131072):
        for ratio in (0.01, 0.05, 0.10, 0.25, 0.5, 1.0):
            assert kvr.kvr_paper_storage_split(N, ratio) == orc.paper_split(N, ratio), (N, ratio)
    assert kvr.kvr_paper_storage_split(2048, 0.10) == (184, 92, 7)
    with pytest.raises(kvr.KvrError):
        kvr.kvr_paper_storage_split(0, 0.1)
    with pytest.raises(kvr.KvrError):
        kvr.kvr_paper_storage_split(100, 0.0)


def test_layer_budgets_match_the_oracle():
    import numpy as np
    import pytest
    import paper_2512_17917_b200 as kvr
    from oracle import kvr_oracle as orc
    rng = np.random.default_rng(7)
    for L, N, ratio in ((32, 32768, 0.25), (36, 8192, 0.10), (3, 100, 0.5), (8, 2048, 0.9)):
        for _ in range(5):
            w = (rng.random(L) ** 3 * 10).tolist()
            assert kvr.kvr_layer_budgets(w, N, ratio) == orc.layer_budgets(w, N, ratio)
    assert kvr.kvr_layer_budgets([100.0, 1.0, 1.0], 100, 0.5) == [100, 25, 25]
    with pytest.raises(kvr.KvrError):
        kvr.kvr_layer_budgets([0.0, 0.0], 100, 0.5)
    with pytest.raises(kvr.KvrError):
        kvr.kvr_layer_budgets([1.0, -1.0], 100, 0.5)
