"""GPU parity of the per-token loss call (rl_token_loss, through the C ABI) against the float64 oracle on the
same seeded fp32 inputs.  The kernel computes each token's terms in fp32 (two exponentials, a handful of
multiplications) and sums in double, so the bars are far inside the path's own: loss 1e-5 relative, derivatives
5e-6 relative element by element (plus 1e-6 of the largest entry, for tokens whose surrogate and KL parts cancel), clip fraction and valid count exact.  The clip decision is taken in fp32 on the
device and in fp64 in the oracle: a token whose ratio lies within 1e-5 of a clip boundary gets old_logp = logp."""
import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2512_21450_b200 import Context
    c = Context(0)
    yield c
    c.close()


def _np64(t):
    return t.detach().double().cpu().numpy()


def _case(seed, T, p_valid=0.6, sigma_old=0.3):
    rng = np.random.default_rng(seed)
    logp = (-4.0 + rng.normal(size=T) * 1.5).astype(np.float32)
    np.minimum(logp, -1e-3, out=logp)
    old = (logp + rng.normal(size=T) * sigma_old).astype(np.float32)
    ref = (logp + rng.normal(size=T) * 0.2).astype(np.float32)
    ent = rng.uniform(0.0, 11.9, size=T).astype(np.float32)
    adv = rng.normal(size=T).astype(np.float32)
    adv[rng.random(T) < 0.1] = 0.0                     # zero-variance groups
    mask = (rng.random(T) < p_valid).astype(np.uint8)
    return logp, ent, old, ref, adv, mask


def _check(ctx, arrays, eps_low, eps_high, beta, ent_coef, use_mask=True, weights=None, offset=0):
    logp, ent, old, ref, adv, mask = arrays
    T = logp.size
    rho = np.exp(logp.astype(np.float64) - old.astype(np.float64))
    near = np.minimum(np.abs(rho - (1 - eps_low)), np.abs(rho - (1 + eps_high))) < 1e-5
    old = np.where(near, logp, old)        # a ratio on a clip boundary becomes 1: same decision on both sides

    def dev(a):
        # an optional element offset makes every array start off a 16-byte boundary (scalar path of the kernel)
        if a is None:
            return None
        buf = torch.empty(a.size + 4, dtype=torch.from_numpy(a).dtype, device="cuda")
        view = buf[offset:offset + a.size]
        view.copy_(torch.from_numpy(a))
        return view

    m = mask if use_mask else None
    o = O.token_loss(logp, ent if ent_coef else None, old, ref if beta else None, adv, m, eps_low, eps_high, beta,
                     ent_coef=ent_coef, token_weight=weights)
    pre = {k: torch.full((T + 4,), float("nan"), device="cuda")[offset:offset + T] for k in ("dlogp", "dentropy")}
    out = ctx.rl_token_loss(dev(logp), dev(ent) if ent_coef else None, dev(old), dev(ref) if beta else None, dev(adv),
                            dev(m), eps_low, eps_high, beta, ent_coef=ent_coef, token_weight=dev(weights), out=pre)
    assert ctx.last_device_status()[0] == 0
    assert abs(out["loss"].item() - o["loss"]) <= 1e-5 * abs(o["loss"]) + 1e-9
    for k in ("dlogp", "dentropy"):
        got = _np64(out[k])
        assert np.isfinite(got).all()
        # the two parts of d loss / d logp (surrogate, KL) may cancel: a floor of 1e-6 of the largest entry
        assert np.all(np.abs(got - o[k]) <= 5e-6 * np.abs(o[k]) + 1e-6 * np.abs(o[k]).max() + 1e-12), k
        if use_mask:
            assert not got[mask == 0].any()
    met = _np64(out["metrics"])
    n_valid = int(mask.sum()) if use_mask else T
    want = [o["pg_loss"], o["kl_mean"], o["entropy_mean"] if ent_coef else 0.0, o["clip_frac"], o["ratio_mean"], o["ratio_max"]]
    for g, w_ in zip(met[:6], want):
        assert abs(g - w_) <= 1e-5 * abs(w_) + 1e-7
    assert met[6] == n_valid and met[7] == 0.0
    return out


@pytest.mark.parametrize("T", [1, 3, 4, 5, 1023, 1024, 4099, 300001])
def test_token_loss_matches_oracle(ctx, T):
    arrays = _case(1000 + T, T)
    if T <= 5:
        arrays[5][:] = 1
    _check(ctx, arrays, 0.2, 0.2, 0.04, 0.0)
    _check(ctx, arrays, 0.2, 0.28, 0.0, 1e-3)                 # asymmetric clip, no KL term, entropy bonus
    _check(ctx, arrays, 0.1, 0.3, 0.5, 0.01, use_mask=False)  # no mask: every row valid
    _check(ctx, arrays, 0.2, 0.2, 0.04, 0.0, offset=1)        # arrays off the 16-byte boundary


def test_token_loss_weights_count_and_degenerate_cases(ctx):
    T = 5000
    arrays = _case(77, T)
    logp, ent, old, ref, adv, mask = arrays
    rng = np.random.default_rng(3)
    w = rng.uniform(0.0, 2.0 / T, size=T).astype(np.float32)
    _check(ctx, arrays, 0.2, 0.2, 0.04, 0.02, weights=w)
    # a caller-supplied divisor of the token mean (data-parallel global count): every term scales by n_valid / count
    t = lambda a: torch.from_numpy(a).cuda()  # noqa: E731
    count = torch.tensor([3 * int(mask.sum())], dtype=torch.int64, device="cuda")
    base = ctx.rl_token_loss(t(logp), t(ent), t(old), t(ref), t(adv), t(mask), 0.2, 0.2, 0.04, 0.02)
    third = ctx.rl_token_loss(t(logp), t(ent), t(old), t(ref), t(adv), t(mask), 0.2, 0.2, 0.04, 0.02, token_count=count)
    assert abs(third["loss"].item() * 3 - base["loss"].item()) <= 1e-6 * abs(base["loss"].item())
    assert torch.allclose(third["dlogp"] * 3, base["dlogp"], rtol=1e-6, atol=0)
    assert third["metrics"][6].item() == int(mask.sum())
    # nothing valid: zero loss, zero derivatives; no rows: zero loss
    none = ctx.rl_token_loss(t(logp), t(ent), t(old), t(ref), t(adv), torch.zeros(T, dtype=torch.uint8, device="cuda"),
                             0.2, 0.2, 0.04, 0.02)
    assert none["loss"].item() == 0.0 and not none["dlogp"].any() and not none["dentropy"].any()
    e = torch.empty(0, device="cuda")
    empty = ctx.rl_token_loss(e, None, e, None, e, None, 0.2, 0.2, 0.0)
    assert empty["loss"].item() == 0.0 and not empty["metrics"].any()
    # two calls give the same bits (fixed-order reduction)
    again = ctx.rl_token_loss(t(logp), t(ent), t(old), t(ref), t(adv), t(mask), 0.2, 0.2, 0.04, 0.02)
    assert again["loss"].item() == base["loss"].item() and torch.equal(again["dlogp"], base["dlogp"])


def test_token_loss_argument_errors(ctx):
    from paper_2512_21450_b200.binding import RLHeadError
    x = torch.zeros(8, device="cuda")
    for kw in (dict(eps_low=1.0), dict(eps_high=-0.1), dict(beta=-1.0), dict(ent_coef=-1.0)):
        a = dict(eps_low=0.2, eps_high=0.2, beta=0.0, ent_coef=0.0)
        a.update(kw)
        with pytest.raises(RLHeadError):
            ctx.rl_token_loss(x, x, x, x, x, None, a["eps_low"], a["eps_high"], a["beta"], ent_coef=a["ent_coef"])
    with pytest.raises(RLHeadError):
        ctx.rl_token_loss(x, None, x, None, x, None, 0.2, 0.2, 0.04)      # beta > 0 without ref_logp
    with pytest.raises(RLHeadError):
        ctx.rl_token_loss(x, None, x, x, x, None, 0.2, 0.2, 0.04, ent_coef=0.1)   # entropy bonus without entropies
    assert ctx.last_device_status()[0] == 0


def test_token_loss_agrees_with_the_fused_path(ctx):
    # the fused call's own log-probabilities and entropies, fed to the per-token call, give the fused call's loss
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(0, device="cuda:0")
    _, adv_tok = ctx.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
    full = ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask, w.eps_low, w.eps_high,
                                      w.beta)
    part = ctx.rl_token_loss(full["logp"], full["entropy"], w.old_logp, w.ref_logp, adv_tok, w.mask, w.eps_low,
                             w.eps_high, w.beta)
    assert abs(part["loss"].item() - full["loss"].item()) <= 1e-6 * abs(full["loss"].item()) + 1e-9
    assert torch.allclose(part["metrics"][:7], full["metrics"][:7], rtol=1e-6, atol=1e-9)
