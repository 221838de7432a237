"""tj_td_error_static: the TD-error call for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is forbidden: inside a latency-critical loop (an allocation
synchronises the device), under a memory plan fixed at start-up, or as a guest of another framework's
allocator.  For them the library keeps the reduction scratch in a fixed array of its own.  This test calls
that entry point through the C ABI twice in a row and requires the same numbers as tj_td_error gives, and
checks that an oversized batch is refused with a message that names the limit.  It lives in the file pytest
collects last so that a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest

from parity_util import RTOL_FP32, blob_for, fields_for

pytestmark = pytest.mark.gpu


def test_td_error_static_matches_td_error_on_two_calls_in_a_row():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2502_20190_b200 import binding as b, build
    build.build()
    f = fields_for(env_kind=0, n_envs=64, obs_dim=4, n_actions=2, hidden=64, epsilon=0.1, seed=31337,
                   replay_capacity=64 * 32, minibatch=1000, staleness_bound=8, warmup=64, target_sync_interval=2,
                   gamma=0.99, huber_delta=1.0)
    ctx = b.Context(**f)
    batch = ctx.alloc_batch()
    dev = ctx.device
    for call in range(2):                      # two calls in a row: the shared scratch keeps the last call's contents
        ctx.publish_weights(blob_for(f, call + 1))
        ctx.actor_step(8)
        ctx.replay_sample(batch=batch)
        ref = ctx.td_error(batch)
        td = torch.full((1000,), float("nan"), device=dev)
        hub = torch.full((1000,), float("nan"), device=dev)
        loss = torch.full((1,), float("nan"), device=dev)
        st = b.tj_td_error_static(ctx.h, batch["c"], td.data_ptr(), hub.data_ptr(), loss.data_ptr())
        assert st == b.TJ_OK, b.tj_last_error(ctx.h)
        torch.cuda.synchronize()
        for got, want in ((td, ref["td"]), (hub, ref["huber"]), (loss, ref["loss"])):
            g, w = got.cpu().numpy().astype(np.float64), want.cpu().numpy().astype(np.float64)
            assert np.all(np.isfinite(g))
            assert np.all(np.abs(g - w) <= RTOL_FP32 * (np.abs(w) + np.sqrt(np.mean(w * w))))
    # beyond the stated maximum the call is refused on the host, before anything is launched
    big = ctx.alloc_batch(65537)
    st = b.tj_td_error_static(ctx.h, big["c"], 0, 0, 0)
    assert st == b.TJ_ERR_INVALID_ARG and "65536" in b.tj_last_error(ctx.h)
    assert ctx.stats()["device_error"] == 0
