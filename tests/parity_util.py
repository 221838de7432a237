"""Helpers for the GPU-vs-oracle parity tests (no arithmetic of the method lives here)."""
import math

import numpy as np

from paper_2502_20190_b200 import synth

RTOL_FP32 = 1e-5      # relative tolerance for FP32 results
RTOL_BF16 = 2e-2      # relative tolerance for bfloat16 tensor-core layers
MARGIN_FACTOR = 8.0   # a threshold decision is compared exactly when the oracle's margin exceeds this * rtol


def close(g, o, rtol, what=""):
    """|g - o| <= rtol * |o| + rtol * rms(o), element by element."""
    g = np.asarray(g, np.float64)
    o = np.asarray(o, np.float64)
    assert g.shape == o.shape, (what, g.shape, o.shape)
    if o.size == 0:
        return
    rms = math.sqrt(float(np.mean(o * o)))
    err = np.abs(g - o)
    bound = rtol * np.abs(o) + rtol * rms + 1e-30
    bad = err > bound
    assert not bad.any(), "%s: %d of %d outside tolerance, worst |diff|=%.3e at bound %.3e" % (
        what, int(bad.sum()), o.size, float(err[bad].max()), float(bound[bad][np.argmax(err[bad])]))


def angle_close(g, o, rtol, what=""):
    d = (np.asarray(g, np.float64) - np.asarray(o, np.float64) + math.pi) % (2 * math.pi) - math.pi
    assert np.all(np.abs(d) <= rtol * (np.abs(o) + math.pi)), (what, float(np.abs(d).max()))


def fields_for(name=None, **overrides):
    base = synth.WORKLOADS[name] if name else {}
    return synth.config_fields(base, **overrides)


def make_pair(orc, binding, **fields):
    """(gpu context, oracle) built from the same configuration fields."""
    ctx = binding.Context(**fields)
    o = orc.Oracle(**fields)
    return ctx, o


def blob_for(fields, version, seed=None):
    vh = fields.get("policy_kind", 0) == 1
    return synth.policy_blob(fields["seed"] if seed is None else seed, version, fields["obs_dim"], fields["hidden"],
                             fields["n_actions"], vh, bf16_exact=False)


REPORT = []          # lines the terminal summary prints after the run (tests/conftest.py)


class Tally:
    """Counts decisions that fell inside the oracle's margin (compared for validity, not equality)."""

    def __init__(self):
        self.total = 0
        self.ambiguous_done = 0
        self.ambiguous_act = 0
        self.max_logit_dev = 0.0      # largest |GPU - oracle| network output seen, relative to the oracle's rms

    def report(self, name):
        """Record the shares of decisions that fell inside a margin: they are counted and shown, never dropped silently."""
        n = max(self.total, 1)
        line = "%s: %d decisions, ambiguous actions %.3f %%, ambiguous done flags %.3f %%, largest output deviation %.2e of rms" % (
            name, self.total, 100.0 * self.ambiguous_act / n, 100.0 * self.ambiguous_done / n, self.max_logit_dev)
        REPORT.append(line)
        print(line)
        return self.ambiguous_act / n, self.ambiguous_done / n


def measured_margin(g_logits, o_logits):
    """Twice the largest deviation between the two sides' outputs on this step.  When the oracle's gap between its two
    largest outputs exceeds it, both sides must pick the same maximum whatever the rounding: a margin taken from what
    was measured, not from the tolerance (which the outputs are checked against separately)."""
    return 2.0 * float(np.max(np.abs(np.asarray(g_logits, np.float64) - np.asarray(o_logits, np.float64)))) + 1e-12


def lockstep_step(ctx, o, torch, *, rtol, env_kind, tally, logits_exact=None, act_rtol=None, dbg=None):
    """Copy the GPU's state into the oracle, advance both by one step, compare everything the step produced.

    The FP32 MLP has one rounding order on both sides, so its outputs are compared bit for bit whenever the
    observation itself is bit-identical (CartPole, LinGauss: the state).  Acrobot's observation goes through
    sin/cos, whose last bit differs between libraries, so there the outputs are compared within tolerance."""
    if logits_exact is None:
        logits_exact = env_kind != 1
    N, D, A = ctx.N, ctx.D, ctx.A
    st = ctx.get_state()
    s0 = st["state"].cpu().numpy()
    ep0 = st["ep_step"].cpu().numpy()
    o.state[:] = s0
    o.ep_step[:] = ep0
    o.set_counters(st["cursor"], st["t"], st["k"])
    if dbg is None:
        dbg = torch.empty((N, A), dtype=torch.float32, device=ctx.device)
    ctx.actor_step(1, dbg)
    assert o.actor_step(1) == 0
    g_logits = dbg.cpu().numpy()
    o_logits = o.last("logits")
    if logits_exact:
        assert np.array_equal(g_logits.view(np.uint32), o_logits.view(np.uint32)), "logits differ bitwise"
    else:
        close(g_logits, o_logits, rtol, "logits")
        rms = math.sqrt(float(np.mean(o_logits.astype(np.float64) ** 2))) + 1e-30
        tally.max_logit_dev = max(tally.max_logit_dev, float(np.max(np.abs(g_logits.astype(np.float64) - o_logits))) / rms)
    st1 = ctx.get_state()
    g_state = st1["state"].cpu().numpy()
    g_ep = st1["ep_step"].cpu().numpy()
    o_done = o.last("done").copy()
    o_act = o.last("act").copy()
    dmargin = o.last("done_margin")
    amargin = o.last("act_margin")
    tally.total += N
    on_policy = ctx.cfg.replay_capacity == 0
    if not on_policy:
        ring, block_ver = ctx.ring_view()
        C_ = ctx.cfg.replay_capacity
        base = st["cursor"] % C_
        g_rec = ring[base:base + N].cpu().numpy()
        o_rec = o.ring[base:base + N]
        gi, oi = g_rec.view(np.int32), o_rec.view(np.int32)
        g_act, g_done, g_ver = gi[:, 2 * D], gi[:, 2 * D + 2], gi[:, 2 * D + 3]
        assert np.array_equal(g_ver, oi[:, 2 * D + 3]), "version tags differ"
        assert int(block_ver[base // N].item()) == int(o.block_version[base // N])
        g_rew, g_obs, g_next = g_rec[:, 2 * D + 1], g_rec[:, :D], g_rec[:, D:2 * D]
        o_rew, o_obs, o_next = o_rec[:, 2 * D + 1], o_rec[:, :D], o_rec[:, D:2 * D]
    else:
        g_act = g_done = g_rew = g_obs = g_next = None
    words = None
    if ctx.cfg.policy_kind == 0:
        import oracle as _orc
        thr = _orc.explore_threshold(ctx.cfg.epsilon)
        words = (thr, [_orc.stream_words(ctx.cfg.seed, 0, 0, e, st["t"]) for e in range(N)])
    return dict(words=words, st=st, st1=st1, g_state=g_state, g_ep=g_ep, g_logits=g_logits, o_logits=o_logits, o_done=o_done,
                o_act=o_act, dmargin=dmargin, amargin=amargin, g_act=g_act, g_done=g_done, g_rew=g_rew, g_obs=g_obs,
                g_next=g_next, o_rew=None if on_policy else o_rew, o_obs=None if on_policy else o_obs,
                o_next=None if on_policy else o_next, s0=s0, ep0=ep0)


def compare_ring_step(r, o, *, rtol, env_kind, tally, act_exact=True, act_margin_scale=None):
    """Checks on the records, actions, done flags and next states of one lockstep step (ring mode)."""
    N = r["g_state"].shape[0]
    # actions: exact, except inside the oracle's greedy margin when the logits are only close; and the GPU's
    # own outputs, pushed through the oracle's selection rule with the same Philox words, must give its action
    if r["words"] is not None:
        import oracle as _orc
        thr, words = r["words"]
        mine = np.array([_orc.select_eps_greedy(r["g_logits"][e], words[e][0], words[e][1], thr) for e in range(N)])
        assert np.array_equal(mine, r["g_act"]), "selection rule differs on the GPU's own outputs"
    if act_exact:
        assert np.array_equal(r["g_act"], r["o_act"]), "actions differ"
        act_ok = np.ones(N, bool)
    else:
        sure = r["amargin"] > act_margin_scale
        assert np.array_equal(r["g_act"][sure], r["o_act"][sure]), "actions differ outside the decision margin"
        act_ok = r["g_act"] == r["o_act"]
        tally.ambiguous_act += int((~sure).sum())
    # done: exact outside the threshold margin
    sure_d = r["dmargin"] > MARGIN_FACTOR * rtol
    assert np.array_equal(r["g_done"][sure_d & act_ok], r["o_done"][sure_d & act_ok]), "done flags differ"
    tally.ambiguous_done += int((~sure_d).sum())
    same = act_ok & (r["g_done"] == r["o_done"])
    # record payload
    if env_kind == 0:
        assert np.array_equal(r["g_obs"], r["o_obs"])           # the observation is the state itself
    else:
        close(r["g_obs"], r["o_obs"], rtol, "obs")
    close(r["g_next"][same], r["o_next"][same], rtol, "next_obs")
    close(r["g_rew"][same], r["o_rew"][same], rtol, "reward")
    # state after the step: fresh draws are bit-exact, stepped states within tolerance
    g_state, o_state = r["g_state"], o.state
    was_done = same & (r["o_done"] != 0)
    assert np.array_equal(g_state[was_done], o_state[was_done]), "reset states differ"
    cont = same & (r["o_done"] == 0)
    if env_kind == 1:
        angle_close(g_state[cont][:, :2], o_state[cont][:, :2], rtol, "angles")
        close(g_state[cont][:, 2:], o_state[cont][:, 2:], rtol, "velocities")
    else:
        close(g_state[cont], o_state[cont], rtol, "state")
    assert np.array_equal(r["g_ep"][same], o.ep_step[same])
