"""tj_td_error_static: the TD-error call for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is forbidden: inside a latency-critical loop (an allocation
synchronises the device), under a memory plan fixed at start-up, or as a guest of another framework's
allocator.  For them the library keeps the reduction scratch in a fixed array of its own.  This test calls
that entry point through the C ABI twice in a row and requires the same numbers as tj_td_error gives (and as the
CPU oracle gives for the same rows), and checks that an oversized batch is refused with a message that names the
limit.  A second test covers a bfloat16 context, where this entry point runs the FP32 kernels on the rounded
weights while tj_td_error uses the tensor cores.  It lives in the file pytest collects last so that a failure here
cannot hide the result of any other test.
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
    import oracle
    build.build()
    oracle.build()
    f = fields_for(env_kind=0, n_envs=64, obs_dim=4, n_actions=2, hidden=64, epsilon=0.1, seed=31337,
                   replay_capacity=64 * 32, minibatch=1000, staleness_bound=8, warmup=64, target_sync_interval=2,
                   gamma=0.99, huber_delta=1.0)
    ctx = b.Context(**f)
    orc = oracle.Oracle(**dict(f, n_envs=4, replay_capacity=16, minibatch=4, warmup=0))
    batch = ctx.alloc_batch()
    dev = ctx.device
    launches = ctx.stats()["kernel_launches"]
    for call in range(2):                      # two calls in a row: the shared scratch keeps the last call's contents
        ctx.publish_weights(blob_for(f, call + 1))
        orc.publish(blob_for(f, call + 1))     # target stays at the first version on both sides (no learner step yet / interval 2)
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
        # and against the oracle, row by row
        rec = np.zeros((1000, 12), np.float32)
        rec[:, :4] = batch["obs"].cpu().numpy()
        rec[:, 4:8] = batch["next_obs"].cpu().numpy()
        rec.view(np.int32)[:, 8] = batch["act"].cpu().numpy()
        rec[:, 9] = batch["rew"].cpu().numpy()
        rec.view(np.int32)[:, 10] = batch["done"].cpu().numpy()
        ost, o_td, o_hub, o_loss, qs, qn = orc.td(rec)
        assert ost == 0
        terms = np.abs(qs) + np.abs(qn) + np.abs(rec[:, 9])
        assert np.all(np.abs(td.cpu().numpy() - o_td) <= RTOL_FP32 * (np.abs(o_td) + terms))
        assert abs(float(loss.item()) - o_loss) <= 2 * RTOL_FP32 * (abs(o_loss) + float(terms.mean()))
        orc.set_counters(0, 0, call + 1)       # the GPU side took one learner step (its sample call)
    # beyond the stated maximum the call is refused on the host, before anything is launched
    big = ctx.alloc_batch(65537)
    st = b.tj_td_error_static(ctx.h, big["c"], 0, 0, 0)
    assert st == b.TJ_ERR_INVALID_ARG and "65536" in b.tj_last_error(ctx.h)
    s = ctx.stats()
    assert s["device_error"] == 0
    # launches counted: per call 1 publish + 1 actor + 2 sample + 2 tj_td_error + 2 static; the refused call counts nothing
    assert s["kernel_launches"] - launches == 2 * 8


def test_td_error_static_in_a_bf16_context():
    """In a bfloat16 context tj_td_error runs both forwards on the tensor cores (activations rounded to bfloat16 on the
    way), while the no-allocation variant runs the FP32 kernels on the same rounded weights.  Both must agree with the
    oracle (rounded weights, double accumulation): the FP32 kernels to FP32 accuracy, the tensor-core path to 2e-2."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2502_20190_b200 import binding as b, build, synth
    import oracle
    build.build()
    oracle.build()
    D, H, A, n = 128, 128, 16, 300
    f = fields_for(env_kind=2, n_envs=64, obs_dim=D, n_actions=A, hidden=H, epsilon=0.1, seed=2718, weight_dtype=1,
                   replay_capacity=64 * 16, minibatch=n, staleness_bound=8, warmup=64, target_sync_interval=1000,
                   gamma=0.99, huber_delta=1.0, max_episode_steps=5, lg_done_norm=9.0)
    ctx = b.Context(**f)
    orc = oracle.Oracle(**dict(f, n_envs=4, replay_capacity=16, minibatch=4, warmup=0))
    batch = ctx.alloc_batch()
    dev = ctx.device
    for call in range(2):
        blob = blob_for(f, call + 1)
        ctx.publish_weights(blob)
        orc.publish(blob)
        ctx.actor_step(6)
        ctx.replay_sample(batch=batch)
        tc = ctx.td_error(batch)
        td = torch.full((n,), float("nan"), device=dev)
        hub = torch.full((n,), float("nan"), device=dev)
        loss = torch.full((1,), float("nan"), device=dev)
        assert b.tj_td_error_static(ctx.h, batch["c"], td.data_ptr(), hub.data_ptr(), loss.data_ptr()) == b.TJ_OK
        torch.cuda.synchronize()
        rec = np.zeros((n, 2 * D + 4), np.float32)
        rec[:, :D] = batch["obs"].cpu().numpy()
        rec[:, D:2 * D] = batch["next_obs"].cpu().numpy()
        rec.view(np.int32)[:, 2 * D] = batch["act"].cpu().numpy()
        rec[:, 2 * D + 1] = batch["rew"].cpu().numpy()
        rec.view(np.int32)[:, 2 * D + 2] = batch["done"].cpu().numpy()
        ost, o_td, o_hub, o_loss, qs, qn = orc.td(rec)
        assert ost == 0
        terms = np.abs(qs) + np.abs(qn) + np.abs(rec[:, 2 * D + 1])
        g = td.cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(g))
        assert np.all(np.abs(g - o_td) <= 4 * RTOL_FP32 * (np.abs(o_td) + terms))          # FP32 kernels, rounded weights
        assert abs(float(loss.item()) - o_loss) <= 4 * RTOL_FP32 * (abs(o_loss) + float(terms.mean()))
        q_scale = np.sqrt(np.mean(qs ** 2) + np.mean(qn ** 2))
        g_tc = tc["td"].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(g_tc - o_td) <= 2e-2 * (np.abs(qs) + np.abs(qn) + 2 * q_scale))  # tensor-core path
        assert np.all(np.abs(g_tc - g) <= 2e-2 * (np.abs(qs) + np.abs(qn) + 2 * q_scale))
    assert ctx.stats()["device_error"] == 0
