"""The pins must be able to fail: every plausible mistake planted in a copy of the oracle (a
dropped term, a wrong sign, a wrong divisor, a wrong branch) has to trip at least one pin test.
The mistakes are planted in the oracle's source on the CPU; the real module is untouched."""
import os
import types

import pytest

import tests.test_oracle_pins as pins

ORACLE_SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle", "grpo_oracle.py")

MUTANTS = {
    "entropy sign": ("ent = -(P * LP).sum(axis=1)", "ent = (P * LP).sum(axis=1)"),
    "lse without the max shift added back": ("lse = M[:, 0] + np.log(", "lse = np.log("),
    "k3 constant term dropped": ("k3 = np.exp(delta) - delta - 1.0\n        dk3", "k3 = np.exp(delta) - delta\n        dk3"),
    "k3 gradient sign": ("dk3 = 1.0 - np.exp(delta)          # d k3 / d logp", "dk3 = np.exp(delta) - 1.0"),
    "clip branch ignores the advantage sign": ("active = (rho * adv <= clipped * adv)", "active = (rho <= clipped)"),
    "surrogate not pessimistic": ("s = np.minimum(rho * adv, clipped * adv)\n        # the unclipped",
                                  "s = np.maximum(rho * adv, clipped * adv)\n        # the unclipped"),
    "logit gradient sign": ("G = wdlogp[:, None] * (onehot - P)", "G = wdlogp[:, None] * (P - onehot)"),
    "entropy gradient misses the +Ent term": ("G += (wr * ent_coef)[:, None] * P * (LP + ent[:, None])\n    if kl_full", "G += (wr * ent_coef)[:, None] * P * LP\n    if kl_full"),
    "dW uses the wrong operand": ('out["dW"] = G.T @ Hr', 'out["dW"] = G.T @ (Hr * 0 + 1)'),
    "dH scaled": ('out["dH"][rows] = G @ W ', 'out["dH"][rows] = 2 * G @ W '),
    "population instead of sample variance": ("/ (group_size - ddof)", "/ group_size"),
    "advantage not centred": ("(grp - mu) / (sigma + eps_std)", "grp / (sigma + eps_std)"),
    "token mean divides by all rows": ("return m / n if n > 0", "return m / m.size if n > 0"),
    "sequence ratio sums instead of averaging": ("(logp[idx] - old_logp[idx]).sum() / idx.size", "(logp[idx] - old_logp[idx]).sum()"),
    "per-response mean forgets the number of responses": ("w[sl] = m[sl] / (B * n)", "w[sl] = m[sl] / n"),
    "sequence-level gradient forgets 1/len": ("-(rho / np.maximum(len_full[rows], 1.0)) * seq_sum[rows]", "-rho * seq_sum[rows]"),
    "RLOO includes the response itself": ("if j != i]", "]"),
    "OPO baseline unweighted": ("base = (ln[sl] * r[sl]).sum() / tot", "base = r[sl].sum() / len(r[sl])"),
    "full KL gradient misses the -KL term": ("P * (LP - LQ - kl_full[:, None])", "P * (LP - LQ)"),
    "full KL direction swapped": ("return (np.exp(LP) * (LP - LQ)).sum(axis=1)", "return (np.exp(LQ) * (LQ - LP)).sum(axis=1)"),
    "slice merge forgets to rescale by exp(M_s - M)": ("S = (st[:, t, 1] * np.exp(st[:, t, 0] - M)).sum()", "S = st[:, t, 1].sum()"),
    "slice statistics: weighted sum uses shifted logits": ("stats[t] = (M, e.sum(), (e * z).sum(),", "stats[t] = (M, e.sum(), (e * (z - M)).sum(),"),
    "slice statistics: target id not made local": ("y = int(tokens[t]) - int(vocab_offset)", "y = int(tokens[t])"),
    "slice backward: one-hot not made local": ("y = tokens[rows] - int(vocab_offset)", "y = tokens[rows]"),
    "slice backward: softmax renormalised inside the slice": ("LP = H[rows] @ W_shard.T - np.asarray(lse, dtype=np.float64)[rows][:, None]", "LP = H[rows] @ W_shard.T; LP = LP - np.log(np.exp(LP).sum(axis=1))[:, None]"),
    "shaping: penalty sign": ("shaped[t] = -beta * kl[t]", "shaped[t] = beta * kl[t]"),
    "shaping: trajectory value on the last row instead of the last valid row": ("shaped[valid[-1]] += v[i]", "shaped[int(off[i + 1]) - 1] += v[i]"),
    "shaping: trajectory value dropped": ("shaped[valid[-1]] += v[i]", "pass"),
    "shaping: trajectory value on every token": ("shaped[valid[-1]] += v[i]", "shaped[valid] += v[i]"),
    "shaping: forward instead of reverse cumulative sum": ("for t in reversed(valid):\n            running", "for t in valid:\n            running"),
    "shaping: discount applied to the reward instead of the tail": ("running = shaped[t] + gamma * running", "running = gamma * shaped[t] + running"),
    "shaping: masked rows counted as discount steps": ("valid = [t for t in range(int(off[i]), int(off[i + 1])) if m[t]]\n        if not valid:\n            continue\n        for t in valid:\n            shaped[t] = -beta * kl[t]", "valid = [t for t in range(int(off[i]), int(off[i + 1])) if m[t]]\n        if not valid:\n            continue\n        for t in valid:\n            shaped[t] = -beta * kl[t]\n        valid = list(range(valid[0], valid[-1] + 1))"),
    "shaping: k1 direction swapped": ("return logp - ref\n", "return ref - logp\n"),
    "shaping: k3 uses the opposite log-ratio": ("delta = ref - logp\n        return np.exp(delta) - delta - 1.0", "delta = logp - ref\n        return np.exp(delta) - delta - 1.0"),
    "row map keeps the masked rows": ("return [t for t in range(len(mask)) if mask[t] != 0]", "return [t for t in range(len(mask)) if mask[t] == 0]"),
    "token loss: entropy bonus enters with the wrong sign": ("loss_t = -s + beta * k3 - ent_coef * ent\n    out = dict(", "loss_t = -s + beta * k3 + ent_coef * ent\n    out = dict("),
    "token loss: derivative not weighted": ("dlogp=np.where(rows, w * dlogp, 0.0)", "dlogp=np.where(rows, dlogp, 0.0)"),
    "token loss: entropy derivative sign": ("dentropy=np.where(rows, -w * ent_coef, 0.0)", "dentropy=np.where(rows, w * ent_coef, 0.0)"),
    "token loss: masked rows keep a derivative": ("dlogp=np.where(rows, w * dlogp, 0.0)", "dlogp=dlogp / max(m.sum(), 1.0)"),
    "logits index order": ("return H @ W.T", "return (W @ H.T).T[::-1][::-1] if H.shape[0] == 1 else (H[:, ::-1] @ W[:, ::-1].T if False else H @ W[::-1].T)"),
}

PIN_TESTS = [getattr(pins, n) for n in dir(pins) if n.startswith("test_")]


def _load_mutant(old, new):
    src = open(ORACLE_SRC).read()
    assert src.count(old) >= 1, f"mutation anchor not found: {old!r}"
    mod = types.ModuleType("grpo_oracle_mutant")
    exec(compile(src.replace(old, new), ORACLE_SRC, "exec"), mod.__dict__)
    return mod


def _run_all_pins():
    failures = 0
    for t in PIN_TESTS:
        marks = [m for m in getattr(t, "pytestmark", []) if m.name == "parametrize"]
        cases = [()]
        if marks:
            names, values = marks[0].args
            cases = [v if isinstance(v, tuple) and "," in names else (v,) for v in values]
        for c in cases:
            try:
                t(*c)
            except Exception:          # an assertion, or the mistake breaks the computation outright
                failures += 1
    return failures


def test_unmutated_oracle_passes_every_pin(monkeypatch):
    assert _run_all_pins() == 0


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_is_caught(monkeypatch, name):
    old, new = MUTANTS[name]
    monkeypatch.setattr(pins, "O", _load_mutant(old, new))
    assert _run_all_pins() > 0, f"no pin notices: {name}"
