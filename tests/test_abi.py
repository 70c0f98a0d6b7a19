"""The C-ABI library loads and exports every function its header declares; host-only
entry points (no GPU needed) validate configurations."""
import ctypes
import os
import re

import pytest

from paper_2605_23200_b200 import binding, build, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def test_every_declared_symbol_is_exported():
    header = open(os.path.join(ROOT, "include", "ams.h")).read()
    declared = set(re.findall(r"\b(ams_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS), declared ^ set(binding.EXPORTS)
    lib = binding.lib()
    for name in declared:
        assert getattr(lib, name) is not None


def test_struct_layout_matches_header_order():
    header = open(os.path.join(ROOT, "include", "ams.h")).read()
    body = header[header.index("typedef struct {", header.index("opaque host handle")):header.index("} ams_config;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = []
    for decl in re.findall(r"(?:int32_t|float)\s+([^;]+);", body):
        names += [n.strip() for n in decl.split(",")]
    assert names == [f[0] for f in binding.AmsConfig._fields_]


def test_sizes_and_validation_without_gpu():
    lib = binding.lib()
    for i, wl in inputs.CONFIGS.items():
        cfg = binding.config_for(wl)
        assert lib.ams_ema_state_bytes(ctypes.byref(cfg)) == wl.layers_resident * wl.batch * wl.n_kv_heads * wl.max_seq_len * 4
        assert lib.ams_workspace_bytes(ctypes.byref(cfg)) > 0
        want = wl.n_segments + (2 * (wl.max_seq_len // wl.l_max) if wl.l_max else 0) + 4
        assert lib.ams_segment_capacity(ctypes.byref(cfg)) == want
    cfg = binding.config_for(inputs.CONFIGS[0])
    for field, bad in (("head_dim", 64), ("page_size", 32), ("n_q_heads", 33), ("max_seq_len", 131072 + 16),
                       ("max_seq_len", 1000), ("eps", 0.0), ("ema_lambda", 1.0), ("ema_beta", 1.5), ("max_budget", 0),
                       ("pool_kernel", 0), ("pool_kernel", 4), ("pool_kernel", 65), ("decoupled", 2)):
        c = binding.config_for(inputs.CONFIGS[0])
        setattr(c, field, bad)
        assert lib.ams_workspace_bytes(ctypes.byref(c)) == 0, field
    # a smoothed or separate mass signal costs one more per-token array of workspace
    plain = lib.ams_workspace_bytes(ctypes.byref(cfg))
    per_token = cfg.n_layers * cfg.max_batch * cfg.n_kv_heads * cfg.max_seq_len * 4
    for kw in (dict(pool_kernel=5), dict(decoupled=1), dict(pool_kernel=3, decoupled=1)):
        c = binding.config_for(inputs.CONFIGS[0])
        for k, v in kw.items():
            setattr(c, k, v)
        assert lib.ams_workspace_bytes(ctypes.byref(c)) == plain + per_token
    # the expected-attention scorer keeps one logit per query head and token
    c = binding.config_for(inputs.CONFIGS[0], expected_scorer=1)
    assert lib.ams_workspace_bytes(ctypes.byref(c)) == plain + per_token * (cfg.n_q_heads // cfg.n_kv_heads)
    c.expected_scorer = 2
    assert lib.ams_workspace_bytes(ctypes.byref(c)) == 0
    assert lib.ams_set_query_stats(None, None, None, ctypes.c_float(0.01)) == binding.AMS_ERR_INVALID_ARG
    assert binding.strerror(binding.AMS_ERR_TIMEOUT) == "bounded device wait expired"
    handle = ctypes.c_void_p()
    rc = lib.ams_init_state(ctypes.byref(cfg), None, None, 0, None, ctypes.byref(handle))
    assert rc == binding.AMS_ERR_INVALID_ARG and not handle.value
