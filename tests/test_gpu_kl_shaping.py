"""GPU parity of the token-level KL reward shaping call (rl_kl_shaped_returns, through the C ABI)
against the float64 oracle on the same seeded inputs.  Tolerance: 1e-6 absolute + 1e-6 relative
(sums run in double on the device; the outputs are rounded to fp32 once)."""
import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O

pytestmark = pytest.mark.gpu

TOL = 1e-6


@pytest.fixture(scope="module")
def ctx():
    from paper_2512_21450_b200 import Context
    c = Context(0)
    yield c
    c.close()


def _np64(t):
    return t.detach().double().cpu().numpy()


def _case(seed, lengths, T_extra=0, first=0, p_valid=0.7, value_scale=1.0):
    rng = np.random.default_rng(seed)
    off = np.concatenate([[first], first + np.cumsum(lengths)]).astype(np.int32)
    T = int(off[-1]) + T_extra
    mask = (rng.random(T) < p_valid).astype(np.uint8)
    logp = (-3.0 + rng.normal(size=T) * 0.8).astype(np.float32)
    ref = (logp + rng.normal(size=T) * 0.2).astype(np.float32)
    R = (rng.normal(size=len(lengths)) * value_scale).astype(np.float32)
    kl = rng.random(T).astype(np.float32)
    return off, T, mask, logp, ref, R, kl


def _close(got, want):
    return np.all(np.abs(got - want) <= TOL + TOL * np.abs(want))


@pytest.mark.parametrize("name,lengths,kw", [
    ("short", [5, 1, 17, 32, 33], {}),
    ("ragged_chunks", [31, 64, 65, 127, 128, 129, 300], dict(first=3, T_extra=9)),
    ("empty_ranges", [0, 40, 0, 0, 7, 0], dict(T_extra=2)),
    ("long", [4096, 5000, 1], dict(p_valid=0.7)),
    ("all_masked_response", [50, 60, 70], dict(p_valid=0.0)),
    ("many", [int(x) for x in np.random.default_rng(5).integers(1, 200, size=3000)], dict(first=1)),
])
@pytest.mark.parametrize("kind", ["k1", "k3", "given"])
def test_kl_shaped_returns_match_oracle(ctx, name, lengths, kw, kind):
    off, T, mask, logp, ref, R, kl = _case(sum(map(ord, name)), lengths, **kw)
    if name == "all_masked_response":
        mask[:] = 1
        mask[off[1]:off[2]] = 0
    dev = "cuda"
    t = lambda a: torch.from_numpy(a).to(dev)  # noqa: E731
    for gamma, beta, use_mask in ((1.0, 0.04, True), (0.97, 0.5, True), (1.0, 0.0, False)):
        # the call takes beta and gamma as fp32: both sides get the same (fp32-representable) values
        gamma, beta = float(np.float32(gamma)), float(np.float32(beta))
        sh, ret = ctx.rl_kl_shaped_returns(t(R), t(logp), t(ref), t(mask) if use_mask else None, t(off), T, beta,
                                           gamma=gamma, kind=kind, kl_tok=t(kl),
                                           returns=torch.full((T,), float("nan"), device=dev))
        s, detail = ctx.last_device_status()
        assert s == 0, (s, detail)
        o_sh, o_ret = O.kl_shaped_returns(R.astype(np.float64), logp.astype(np.float64), ref.astype(np.float64),
                                          mask if use_mask else None, off, beta, gamma=gamma, kind=kind,
                                          kl_tok=kl.astype(np.float64))
        if not use_mask:
            o_sh, o_ret = np.pad(o_sh, (0, T - len(o_sh))), np.pad(o_ret, (0, T - len(o_ret)))
        assert not torch.isnan(ret).any() and not torch.isnan(sh).any()
        assert _close(_np64(ret), o_ret), (name, kind, gamma, np.abs(_np64(ret) - o_ret).max())
        assert _close(_np64(sh), o_sh)
        m = mask.astype(bool) if use_mask else np.ones(T, bool)
        assert np.all(_np64(ret)[~m] == 0)
    # the shaped-reward output is optional
    _, ret2 = ctx.rl_kl_shaped_returns(t(R), t(logp), t(ref), t(mask), t(off), T, 0.04, kind=kind, kl_tok=t(kl),
                                       want_shaped=False)
    _, ret3 = ctx.rl_kl_shaped_returns(t(R), t(logp), t(ref), t(mask), t(off), T, 0.04, kind=kind, kl_tok=t(kl))
    assert torch.equal(ret2, ret3)       # fixed summation order: bitwise reproducible


def test_kl_shaped_returns_feed_the_loss(ctx):
    # the shaped returns are per-row advantages of the loss call: workload rows, GRPO advantages as the
    # per-response scalar, k3 shaping from the workload's own old / reference log-probabilities
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(1, prompts=1, L_max=48, d=256, V=3000, seed=811)
    adv_seq = ctx.rl_grpo_advantages(w.rewards, w.G)
    beta = float(np.float32(0.1))
    _, ret = ctx.rl_kl_shaped_returns(adv_seq, w.old_logp, w.ref_logp, w.mask, w.seq_offsets, w.T, beta)
    o_adv = O.grpo_advantages(w.rewards.cpu().numpy(), w.G)
    _, o_ret = O.kl_shaped_returns(o_adv, _np64(w.old_logp), _np64(w.ref_logp), w.mask.cpu().numpy(),
                                   w.seq_offsets.cpu().numpy(), beta)
    assert _close(_np64(ret), o_ret)
    out = ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, None, ret, w.mask, w.eps_low, w.eps_high, 0.0)
    oo = O.policy_loss_fwd_bwd(_np64(w.H), _np64(w.W), w.tokens.cpu().numpy(), _np64(w.old_logp), None, o_ret,
                               w.mask.cpu().numpy(), w.eps_low, w.eps_high, 0.0)
    assert abs(out["loss"].item() - oo["loss"]) <= 1e-3 * abs(oo["loss"]) + 1e-7
    rel = lambda a, b: np.linalg.norm(a - b) / np.linalg.norm(b)  # noqa: E731
    assert rel(_np64(out["dH"]), oo["dH"]) <= 1e-2 and rel(_np64(out["dW"]), oo["dW"]) <= 1e-2


def test_kl_shaped_returns_argument_checks(ctx):
    from paper_2512_21450_b200.binding import RLHeadError
    off, T, mask, logp, ref, R, kl = _case(1, [4, 4])
    t = lambda a: torch.from_numpy(a).cuda()  # noqa: E731
    with pytest.raises(RLHeadError):
        ctx.rl_kl_shaped_returns(t(R), t(logp), t(ref), None, t(off), T, -1.0)
    with pytest.raises(RLHeadError):
        ctx.rl_kl_shaped_returns(t(R), t(logp), t(ref), None, t(off), T, 0.1, gamma=-0.5)
    with pytest.raises(RLHeadError):
        ctx.rl_kl_shaped_returns(t(R), None, t(ref), None, t(off), T, 0.1, kind="k1")
    with pytest.raises(RLHeadError):
        ctx.rl_kl_shaped_returns(t(R), t(logp), t(ref), None, t(off), T, 0.1, kind="given", kl_tok=None)
    # n_seq = 0: everything is outside every range
    _, ret = ctx.rl_kl_shaped_returns(t(R[:0]), t(logp), t(ref), None, t(off[:1]), T, 0.1)
    assert not ret.any()
