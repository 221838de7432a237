"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares, and its
host-side configuration logic answers without touching a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2502_20190_b200 import binding as b
from paper_2502_20190_b200 import build as tjbuild
from paper_2502_20190_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    tjbuild.build()
    return b.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "tj.h")).read()
    declared = set(re.findall(r"^(?:int|const char \*)\s*(tj_[a-z0-9_]+)\s*\(", header, re.M))
    assert declared == set(b.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_config_struct_matches_and_workspace_sizes(lib):
    for name, w in synth.WORKLOADS.items():
        cfg, _keep = b.make_config(**synth.config_fields(w))
        st, nbytes, align = b.tj_query_workspace(cfg)
        assert st == b.TJ_OK and align == 256, (name, b.tj_last_error())
        C_, N, D = w["replay_capacity"], w["n_envs"], w["obs_dim"]
        if C_:
            assert nbytes >= C_ * (2 * D + 4) * 4
            # beside the ring and the env state: the learner update's scratch (four activation / delta arrays of
            # minibatch x hidden, 32 partial gradients of the parameter blob, W2 transposed, the split copies of W1 (two
            # networks), W2 (two) and W2^T for the tensor-core products) and 64 MiB for the rest
            B, H = w["minibatch"], w["hidden"]
            update = (4 * B * H + 32 * (H * (D + H + 19) + 17) + H * H + 24 * B + 2 * (2 * H * D + 3 * H * H)) * 4
            assert nbytes < C_ * (2 * D + 4) * 4 + N * max(D, 4) * 4 + update + 64 * 2**20
    # the largest workload's ring is 16M records of 1040 bytes
    assert nbytes > 17.4e9


@pytest.mark.parametrize("change, status", [
    (dict(struct_size=8), b.TJ_ERR_CONFIG),
    (dict(n_envs=0), b.TJ_ERR_CONFIG),
    (dict(replay_capacity=65537), b.TJ_ERR_CONFIG),     # not a multiple of n_envs
    (dict(obs_dim=5), b.TJ_ERR_CONFIG),
    (dict(n_actions=3), b.TJ_ERR_CONFIG),
    (dict(epsilon=1.5), b.TJ_ERR_CONFIG),
    (dict(policy_kind=1), b.TJ_ERR_CONFIG),             # ring + categorical
    (dict(minibatch=0), b.TJ_ERR_CONFIG),
])
def test_bad_configs_are_refused_on_the_host(lib, change, status):
    cfg, _ = b.make_config(**synth.config_fields(synth.WORKLOADS["cfg1"]))
    for k, v in change.items():
        setattr(cfg, k, v)
    st, _, _ = b.tj_query_workspace(cfg)
    assert st == status and b.tj_last_error()


def test_null_arguments_are_refused(lib):
    cfg, _ = b.make_config(**synth.config_fields(synth.WORKLOADS["cfg1"]))
    assert lib.tj_query_workspace(C.byref(cfg), None, None) == b.TJ_ERR_INVALID_ARG
    assert lib.tj_create(C.byref(cfg), None, 0, None, None) == b.TJ_ERR_INVALID_ARG
    h = C.c_void_p()
    assert lib.tj_create(C.byref(cfg), None, 0, None, C.byref(h)) == b.TJ_ERR_INVALID_ARG
    assert lib.tj_create(C.byref(cfg), 12345, 1 << 30, None, C.byref(h)) == b.TJ_ERR_WORKSPACE  # misaligned
    assert lib.tj_destroy(None) == b.TJ_ERR_INVALID_ARG
    assert lib.tj_actor_step(None, 1, None) == b.TJ_ERR_INVALID_ARG


def test_binding_refuses_to_run_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        b.Context(**synth.config_fields(synth.WORKLOADS["cfg1"]))
