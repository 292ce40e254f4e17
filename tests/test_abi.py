"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2507_23777_b200 import binding, build, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def test_header_symbols_are_exported(lib):
    hdr = open(os.path.join(ROOT, "include", "xsm.h")).read()
    declared = set(re.findall(r"XSM_API[^;(]*?\b(xsm_\w+)\s*\(", hdr))
    assert declared == set(binding.EXPORTS), declared ^ set(binding.EXPORTS)
    raw = ctypes.CDLL(binding.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), name


def test_sizes_and_config_checks(lib):
    for i in range(5):
        cfg = inputs.config(i)
        mc = binding.model_config(cfg)
        assert binding.xsm_weights_bytes(mc) == inputs.n_weight_elements(cfg) * (2 if cfg["dtype"] else 4)
        ws = binding.xsm_workspace_bytes(mc)
        P, K1 = cfg["page_size"], cfg["n_draft"] + 1
        pages = cfg["batch"] * -(-(cfg["max_seq_len"] + K1) // P)
        pool = pages * cfg["n_layers"] * 2 * cfg["d_model"] * P * (2 if cfg["dtype"] else 4)
        assert pool < ws < pool + (2 << 30)
        assert ws < 170e9          # fits one B200
    bad = inputs.config(1)
    bad["d_head"] = 48             # n_heads * d_head != d_model
    assert binding.xsm_weights_bytes(binding.model_config(bad)) == 0
    bad = inputs.config(1, n_draft=17)
    assert binding.xsm_workspace_bytes(binding.model_config(bad)) == 0


def test_null_arguments_are_rejected_on_the_host(lib):
    mc = binding.model_config(inputs.config(0))
    out = ctypes.c_void_p()
    assert lib.xsm_create(ctypes.byref(mc), None, None, 0, None, ctypes.byref(out)) == binding.XSM_ERR_INVALID_ARG
    assert b"null" in lib.xsm_last_error(None)
    assert lib.xsm_spec_step(None, None, None) == binding.XSM_ERR_INVALID_ARG
    assert lib.xsm_destroy(None) == binding.XSM_ERR_INVALID_ARG
    assert lib.xsm_kernel_launches(None) == 0


def test_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    cfg = inputs.config(0)
    with pytest.raises(RuntimeError):
        binding.Context(cfg, inputs.make_weights(cfg))


def test_speedup_formula_reproduces_tables_3_and_4():
    """speedup = SCR * latency(A) / latency(row) (Sec. 5.1) against the printed rows."""
    from paper_2507_23777_b200 import metrics
    rows = [l.split() for l in open(os.path.join(ROOT, "tests", "golden", "table3_table4_speedup.txt")) if l[0] != "#"]
    base = float(rows[0][2])
    assert rows[0][0] == "A" and len(rows) == 7
    for name, scr, lat, printed in rows:
        assert abs(metrics.speedup(float(scr), base, float(lat)) - float(printed)) < 0.011, name


def test_algorithmic_bytes_match_hand_count():
    from paper_2507_23777_b200 import metrics
    a = metrics.algorithmic_bytes(inputs.config(2), 1)      # medium: 24 layers, d 1024, f 4096, V 4096, K 4
    assert a["backbone"] == 24 * (6 * 1024 ** 2 + 3 * 1024 * 4096) * 2 == 905969664
    assert a["fixed"] == 905969664 + 8388608 + 41943040 + 24 * 2 * 257 * 1024 * 2
    assert a["per_position"] == 98304
