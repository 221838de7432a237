"""Full-size workloads in the launch configuration bench.py times (several actor steps per call, then a learner
step and a publish).  The oracle cannot run these sizes, so every check is either on sampled environments and
samples, recomputed one by one from the oracle's building blocks, or a property that holds at any size:
records are self-contained (obs, action, reward, next_obs, done, version), consecutive records of one env chain
(next_obs -> obs, or a reset drawn from Philox), the sampler's indices follow from the version tags, every sampled
batch respects the staleness bound, gathers are bit-exact copies, counters add up.
"""
import numpy as np
import pytest

from parity_util import REPORT, RTOL_FP32, blob_for, close, fields_for

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import oracle
    from paper_2502_20190_b200 import binding, build
    build.build()
    oracle.build()
    return torch, oracle, binding


def _uniform(orc, x, lo, width):
    return np.float32(np.float64(orc.u01(int(x))) * np.float64(np.float32(width)) + np.float64(np.float32(lo)))


def _bf16_round(x):
    """FP32 -> nearest bfloat16 (ties to even), returned as FP32."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def _check_ring_records(orc, f, blobs_by_version, recs, t_of_row, envs, rtol_logits, exact_logits):
    """recs[i][j]: record of sampled env envs[j] written at actor step t_of_row[i].  CartPole / LinGauss only
    (their observation is the state, so a record determines the whole step)."""
    D, H, A = f["obs_dim"], f["hidden"], f["n_actions"]
    thr = orc.explore_threshold(f["epsilon"])
    kind = f["env_kind"]
    n_amb = 0
    for i, t in enumerate(t_of_row):
        for j, e in enumerate(envs):
            rec = recs[i][j]
            ri = rec.view(np.int32)
            obs, nxt = rec[:D], rec[D:2 * D]
            a, rew, done, ver = int(ri[2 * D]), float(rec[2 * D + 1]), int(ri[2 * D + 2]), int(ri[2 * D + 3])
            blob = blobs_by_version[ver]
            w = orc.stream_words(f["seed"], orc.STREAM_ACTION, 0, int(e), int(t))
            if f["weight_dtype"] == 0:
                q = orc.mlp_forward(blob, D, H, A, obs)
                assert a == orc.select_eps_greedy(q, w[0], w[1], thr)          # same FMA order: exact
            else:
                rb = blob.copy()
                o0 = 0
                for n_out, n_in in ((H, D), (H, H), (A, H)):
                    rb[o0:o0 + n_out * n_in] = _bf16_round(rb[o0:o0 + n_out * n_in])
                    o0 += n_out * n_in + n_out
                q = orc.mlp_forward(rb, D, H, A, obs, f64=True).astype(np.float32)
                explore = int(w[0]) < thr
                top = np.sort(q)[::-1]
                if explore or top[0] - top[1] > 8 * rtol_logits * float(np.sqrt(np.mean(q * q))):
                    assert a == orc.select_eps_greedy(q, w[0], w[1], thr)
                else:
                    n_amb += 1
            if kind == 0:
                sn, r, term, margin = orc.cartpole_step(obs, a)
            else:
                noise = np.concatenate([orc.normal4(orc.stream_words(f["seed"], orc.STREAM_NOISE, b, int(e), int(t)))
                                        for b in range(D // 4)])
                sn, r, term, margin = orc.lingauss_step(obs, a, f["lg_A"], f["lg_B"], noise, f.get("lg_noise_std", 0.01),
                                                        f.get("lg_done_norm", 4.0))
            close(nxt, sn, RTOL_FP32, "next_obs")
            assert abs(rew - r) <= RTOL_FP32 * (abs(r) + 1.0)
            if margin > 8 * RTOL_FP32 and not done:
                assert term == 0
            if margin > 8 * RTOL_FP32 and term:
                assert done == 1
            # chaining: the next record's obs is this record's next_obs, or a fresh Philox draw after a done
            if i + 1 < len(t_of_row) and t_of_row[i + 1] == t + 1:
                nobs = recs[i + 1][j][:D]
                if done:
                    lo, wd = (-0.05, 0.1) if kind == 0 else (-0.1, 0.2)
                    want = np.concatenate([[_uniform(orc, x, lo, wd) for x in
                                            orc.stream_words(f["seed"], orc.STREAM_RESET, b, int(e), int(t))]
                                           for b in range(D // 4)]).astype(np.float32)
                    assert np.array_equal(nobs, want)
                else:
                    assert np.array_equal(nobs, nxt)
    return n_amb


def _records_from_batch(b, D, n):
    rec = np.zeros((n, 2 * D + 4), np.float32)
    rec[:, :D] = b["obs"][:n].cpu().numpy()
    rec[:, D:2 * D] = b["next_obs"][:n].cpu().numpy()
    rec.view(np.int32)[:, 2 * D] = b["act"][:n].cpu().numpy()
    rec[:, 2 * D + 1] = b["rew"][:n].cpu().numpy()
    rec.view(np.int32)[:, 2 * D + 2] = b["done"][:n].cpu().numpy()
    return rec


def _check_td_rows(orc, f, blobs, last, n=64):
    """TD errors of the first n rows of the last sampled batch against the oracle, one row at a time.  The oracle only
    needs the two parameter sets, so it is built small; it sees the same publishes in the same cadence (the target
    network stays at version 1: its refresh interval is far beyond these runs)."""
    D = f["obs_dim"]
    # (a context in weight mode 2 runs its learner-side calls on the FP32 kernels: the oracle's FP32 weights are its reference)
    o = orc.Oracle(**dict({k: v for k, v in f.items() if k != "name"}, n_envs=4, replay_capacity=16, minibatch=4, warmup=0,
                          weight_dtype=0 if f["weight_dtype"] == 2 else f["weight_dtype"]))
    for v in range(1, last["v"] + 1):
        o.publish(blobs[v])
    assert last["v"] < f["target_sync_interval"]
    rec = _records_from_batch(last["batch"], D, n)
    st, td, hub, _, qs, qn = o.td(rec)
    assert st == 0
    g = last["out"]["td"][:n].cpu().numpy().astype(np.float64)
    gh = last["out"]["huber"][:n].cpu().numpy().astype(np.float64)
    if f["weight_dtype"] in (0, 2):
        bound = RTOL_FP32 * (np.abs(td) + np.abs(qs) + np.abs(qn) + 1.0)
    else:   # BF16 tensor-core layers: 2e-2 on the scale of the two network outputs the error is a difference of
        bound = 2e-2 * (np.abs(qs) + np.abs(qn) + np.sqrt(np.mean(qs ** 2) + np.mean(qn ** 2)))
    assert np.all(np.abs(g - td) <= bound), float(np.max(np.abs(g - td) / bound))
    assert np.all(np.abs(gh - hub) <= 2 * bound * np.maximum(1.0, np.abs(td)))
    REPORT.append("%s full size: TD error of %d rows vs oracle, worst |diff| / bound = %.3f" % (
        f.get("name", "workload"), n, float(np.max(np.abs(g - td) / bound))))


def _run_ring_workload(env, name, n_iters, sample_envs, sweep=(), weight_dtype=None):
    """The workload's cadence at full size: per iteration one publish, four actor steps in one call, one sample + TD.
    Around it, the staleness side is exercised against a host mirror built from the ring's version tags: a sample with
    bound 0 right after the publish must starve (nothing of the new version exists yet), and every bound of `sweep`
    must give indices that follow from the version tags, batches inside the bound, and counters that add up."""
    torch, orc, binding = env
    f = fields_for(name) if weight_dtype is None else fields_for(name, weight_dtype=weight_dtype)
    ctx = binding.Context(**f)
    f["name"] = name if weight_dtype is None else "%s (weight mode %d)" % (name, weight_dtype)
    N, D, C_, B, S = f["n_envs"], f["obs_dim"], f["replay_capacity"], f["minibatch"], f["staleness_bound"]
    rng = np.random.default_rng(5)
    envs = np.unique(np.concatenate([[0, N - 1, 31, 32], rng.integers(0, N, sample_envs)]))
    blobs = {}
    batch = ctx.alloc_batch()
    ring, block_ver = ctx.ring_view()
    a_steps = 4
    mirror = dict(consumed=0, starved=0, dropped=0, learner_steps=0, max_stale=0, hist=np.zeros(33, np.int64))

    def sample_and_check(bound, v):
        valid = min(ctx.get_state()["cursor"], C_)
        bv = block_ver[:valid // N].cpu().numpy()
        elig = np.nonzero(v - bv <= bound)[0]
        k = ctx.get_state()["k"]
        st, _ = ctx.replay_sample(bound, batch=batch, allow=(0, -7))
        if len(elig) == 0:
            assert st == -7 and ctx.get_state()["k"] == k           # starved: nothing drawn, k unchanged
            mirror["starved"] += 1
            return st
        assert st == 0 and ctx.get_state()["k"] == k + 1
        idx = batch["idx"].cpu().numpy()
        ver = batch["ver"].cpu().numpy()
        assert np.all(v - ver <= bound) and np.all(ver >= 1)         # the staleness invariant, on the whole batch
        assert np.array_equal(ver, bv[idx // N])
        for j in (0, 1, B // 2, B - 1):
            x0 = int(orc.stream_words(f["seed"], orc.STREAM_SAMPLE, 0, j, k)[0])
            r = (x0 * (len(elig) * N)) >> 32
            assert idx[j] == elig[r // N] * N + r % N
        mirror["consumed"] += B
        mirror["learner_steps"] += 1
        mirror["dropped"] += valid - len(elig) * N
        stale = v - ver
        mirror["max_stale"] = max(mirror["max_stale"], int(stale.max()))
        mirror["hist"] += np.bincount(np.minimum(stale, 32), minlength=33)
        return st

    for it in range(n_iters):
        v = it + 1
        blobs[v] = blob_for(f, v)
        assert ctx.publish_weights(blobs[v]) == v
        if it > 0:
            assert sample_and_check(0, v) == -7                     # the consumer is ahead of the producer
        cursor0, t0 = ctx.get_state()["cursor"], ctx.get_state()["t"]
        ctx.actor_step(a_steps)
        for bound in sweep:
            assert sample_and_check(bound, v) == 0
        assert sample_and_check(S, v) == 0
        # gathers are bit-exact copies of the ring rows
        rows = ring[batch["idx"][:64].long()].cpu().numpy()
        assert np.array_equal(batch["obs"][:64].cpu().numpy(), rows[:, :D])
        assert np.array_equal(batch["next_obs"][:64].cpu().numpy(), rows[:, D:2 * D])
        assert np.array_equal(batch["ver"][:64].cpu().numpy(), rows.view(np.int32)[:, 2 * D + 3])
        out = ctx.td_error(batch)
        assert torch.isfinite(out["loss"]).all() and torch.isfinite(out["td"]).all()
        if it == n_iters - 1:
            slots = [[(cursor0 + s * N + int(e)) % C_ for e in envs] for s in range(a_steps)]
            recs = [ring[torch.tensor(sl, device="cuda")].cpu().numpy() for sl in slots]
            last = dict(recs=recs, ts=[t0 + s for s in range(a_steps)], batch=batch, out=out, v=v)
    s = ctx.stats()
    assert s["produced"] == n_iters * a_steps * N and s["device_error"] == 0
    assert s["consumed"] == mirror["consumed"] and s["learner_steps"] == mirror["learner_steps"]
    assert s["starved_calls"] == mirror["starved"] == n_iters - 1
    assert s["dropped_stale"] == mirror["dropped"]
    assert s["actor_steps"] == n_iters * a_steps and sum(s["staleness_hist"]) == s["consumed"]
    assert s["staleness_hist"] == mirror["hist"].tolist()
    assert s["max_sampled_staleness"] == mirror["max_stale"] <= max((S,) + tuple(sweep))
    _check_td_rows(orc, f, blobs, last)
    return ctx, f, blobs, envs, last


def test_cfg2_full_size(env):
    torch, orc, binding = env
    ctx, f, blobs, envs, last = _run_ring_workload(env, "cfg2", n_iters=12, sample_envs=40)
    _check_ring_records(orc, f, blobs, last["recs"], last["ts"], envs, RTOL_FP32, True)


@pytest.mark.parametrize("mode", [0, 2])
def test_cfg3_full_size_single_step_from_state(env, mode):
    """Acrobot: the observation does not determine the state bit for bit, so sampled envs are checked from a
    state snapshot taken before a single step, after the multi-step calls have run.  Weight mode 2 (hidden x hidden layer as
    split-operand tensor-core products) is held to the same tolerance, and its actions to the oracle's wherever the oracle's
    top-2 gap exceeds twice the deviation measured on these rows."""
    torch, orc, binding = env
    ctx, f, blobs, envs, last = _run_ring_workload(env, "cfg3", n_iters=6, sample_envs=30, sweep=(1, 4, 16), weight_dtype=mode)
    N, D, A, H, C_ = f["n_envs"], 6, 3, f["hidden"], f["replay_capacity"]
    st = ctx.get_state()
    s0 = st["state"][torch.tensor(envs, device="cuda")].cpu().numpy()
    dbg = torch.empty((N, A), dtype=torch.float32, device="cuda")
    ctx.actor_step(1, dbg)
    ring, _ = ctx.ring_view()
    slots = [(st["cursor"] + int(e)) % C_ for e in envs]
    recs = ring[torch.tensor(slots, device="cuda")].cpu().numpy()
    logits = dbg[torch.tensor(envs, device="cuda")].cpu().numpy()
    blob = blobs[last["v"]]
    thr = orc.explore_threshold(f["epsilon"])
    qs = np.stack([orc.mlp_forward(blob, D, H, A, orc.acrobot_obs(s0[j])) for j in range(len(envs))])
    margin_q = 2.0 * float(np.max(np.abs(logits.astype(np.float64) - qs))) + 1e-12
    n_in = 0
    for j, e in enumerate(envs):
        obs = orc.acrobot_obs(s0[j])
        q = qs[j]
        close(logits[j], q, RTOL_FP32, "logits")
        w = orc.stream_words(f["seed"], orc.STREAM_ACTION, 0, int(e), int(st["t"]))
        a = int(recs[j].view(np.int32)[2 * D])
        assert a == orc.select_eps_greedy(logits[j], w[0], w[1], thr)
        top = np.sort(q)[::-1]
        if int(w[0]) < thr or top[0] - top[1] > margin_q:
            assert a == orc.select_eps_greedy(q, w[0], w[1], thr)
        else:
            n_in += 1
        sn, r, term, margin = orc.acrobot_step(s0[j], a)
        close(recs[j][:D], obs, RTOL_FP32, "obs")
        close(recs[j][D:2 * D], orc.acrobot_obs(sn), RTOL_FP32, "next_obs")
        if margin > 1e-4:
            assert float(recs[j][2 * D + 1]) == r
    REPORT.append("%s full size: outputs of %d rows within %.2e of rms; %d actions inside the measured margin" % (
        f["name"], len(envs), float(np.max(np.abs(logits - qs))) / float(np.sqrt(np.mean(qs * qs))), n_in))
    assert n_in <= 1


def test_cfg5_full_size_tensor_core_path(env):
    torch, orc, binding = env
    ctx, f, blobs, envs, last = _run_ring_workload(env, "cfg5", n_iters=3, sample_envs=12, sweep=(1, 2, 4, 8, 16))
    n_amb = _check_ring_records(orc, f, blobs, last["recs"], last["ts"], envs, 2e-2, False)
    REPORT.append("cfg5 full size: %d of %d sampled record actions inside the 2e-2 margin" % (n_amb, len(envs) * 4))
    assert n_amb <= 0.3 * len(envs) * 4
    s = ctx.stats()
    # with the literal constants nearly every env terminates on every step
    assert s["episodes_finished"] > 0.9 * s["produced"]
    # one more step at full size with the network outputs exported: sampled rows against the oracle at 2e-2, and the
    # recorded action equal to the oracle's wherever its top-2 gap exceeds twice the deviation measured on these rows
    N, D, H, A, C_ = f["n_envs"], f["obs_dim"], f["hidden"], f["n_actions"], f["replay_capacity"]
    rows = np.unique(np.concatenate([envs, np.arange(0, N, 4099), [127, 128, N - 129, N - 128]]))
    ri = torch.tensor(rows, device="cuda")
    st = ctx.get_state()
    s0 = st["state"][ri].cpu().numpy()
    dbg = torch.empty((N, A), dtype=torch.float32, device="cuda")
    ctx.actor_step(1, dbg)
    g = dbg[ri].cpu().numpy()
    ring, _ = ctx.ring_view()
    acts = ring[((st["cursor"] + ri) % C_).long()][:, 2 * D].view(torch.int32).cpu().numpy()
    rb = blobs[last["v"]].copy()
    o0 = 0
    for n_out, n_in in ((H, D), (H, H), (A, H)):
        rb[o0:o0 + n_out * n_in] = _bf16_round(rb[o0:o0 + n_out * n_in])
        o0 += n_out * n_in + n_out
    q = np.stack([orc.mlp_forward(rb, D, H, A, s0[j], f64=True) for j in range(len(rows))])
    close(g, q, 2e-2, "network outputs at full size")
    margin = 2.0 * float(np.max(np.abs(g - q)))
    thr = orc.explore_threshold(f["epsilon"])
    n_in = 0
    for j, e in enumerate(rows):
        w = orc.stream_words(f["seed"], orc.STREAM_ACTION, 0, int(e), int(st["t"]))
        assert acts[j] == orc.select_eps_greedy(g[j], w[0], w[1], thr)       # the rule, on the GPU's own outputs
        top = np.sort(q[j])[::-1]
        if int(w[0]) < thr or top[0] - top[1] > margin:
            assert acts[j] == orc.select_eps_greedy(q[j].astype(np.float32), w[0], w[1], thr)
        else:
            n_in += 1
    REPORT.append("cfg5 full size: outputs of %d rows within %.2e of rms; %d actions inside the measured margin" % (
        len(rows), float(np.max(np.abs(g - q))) / float(np.sqrt(np.mean(q * q))), n_in))
    assert n_in <= 0.08 * len(rows) + 1
    assert ctx.stats()["device_error"] == 0


@pytest.mark.parametrize("mode", [0, 2])
def test_cfg4_full_size_segments_and_gae(env, mode):
    torch, orc, binding = env
    f = fields_for("cfg4", weight_dtype=mode)
    ctx = binding.Context(**f)
    N, T, D, H, A = f["n_envs"], f["rollout_len"], 4, f["hidden"], 2
    rng = np.random.default_rng(6)
    envs = np.unique(np.concatenate([[0, N - 1], rng.integers(0, N, 10)]))
    blobs = {}
    for seg_i in range(2):
        v = seg_i + 1
        blobs[v] = blob_for(f, v)
        ctx.publish_weights(blobs[v])
        ctx.actor_step(T)
        st, seg = ctx.segment_acquire()
        assert st == 0 and seg["version"] == v
        adv, ret = ctx.gae(seg["rew"], seg["val"], seg["done"], f["gamma"], f["gae_lambda"])
        ei = torch.tensor(envs, device="cuda")
        obs = seg["obs"][:, ei].cpu().numpy()
        act = seg["act"][:, ei].cpu().numpy()
        rew = seg["rew"][:, ei].cpu().numpy()
        done = seg["done"][:, ei].cpu().numpy()
        logp = seg["logp"][:, ei].cpu().numpy()
        val = seg["val"][:, ei].cpu().numpy()
        o_adv, o_ret = orc.gae(rew, val, done, f["gamma"], f["gae_lambda"])
        close(adv[:, ei].cpu().numpy(), o_adv, RTOL_FP32, "adv")
        close(ret[:, ei].cpu().numpy(), o_ret, RTOL_FP32, "ret")
        n_amb = 0
        for t in range(0, T, 9):
            for j, e in enumerate(envs):
                lg, v_ = orc.mlp_forward(blobs[v], D, H, A, obs[t, j], value_head=True)
                if mode == 0:
                    assert val[t, j] == np.float32(v_)                   # same FMA order
                else:
                    assert abs(val[t, j] - v_) <= RTOL_FP32 * (abs(v_) + float(np.sqrt(np.mean(lg * lg) + v_ * v_)))
                u = orc.u01(int(orc.stream_words(f["seed"], orc.STREAM_ACTION, 0, int(e), seg_i * T + t)[0]))
                a, lp, margin = orc.select_categorical(lg, u)
                if margin > 8 * RTOL_FP32:
                    assert act[t, j] == a and abs(logp[t, j] - lp) <= RTOL_FP32 * (abs(lp) + 1)
                else:
                    n_amb += 1
                sn, r, term, m2 = orc.cartpole_step(obs[t, j], int(act[t, j]))
                assert rew[t, j] == r
                if t + 1 < T and not done[t, j]:
                    close(obs[t + 1, j], sn, RTOL_FP32, "chained obs")
        assert n_amb <= 2
    s = ctx.stats()
    assert s["produced"] == 2 * T * N and s["consumed"] == 2 * T * N and s["device_error"] == 0
