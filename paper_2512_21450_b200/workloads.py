"""Seeded synthetic workloads shaped like the paper's 1B-7B VLM GRPO runs.

The paper trains on public datasets that are not needed here: the LM-head path
depends only on shapes, sequence lengths, masks and reward statistics.  This
module fabricates inputs with those properties and nothing else: it serves the
CUDA path and the test oracle alike and contains none of the method's loss or
gradient arithmetic.  The only model-like computation is the stand-in for the
rollout engine and the frozen old/reference policies: tokens are drawn from
softmax(H W^T) by the Gumbel-max trick with torch library ops, and the
"behaviour" and "reference" log-probabilities are that draw's log-probability
plus Gaussian noise.

Workload k uses seed 251221450 + k; lengths, rewards and masked spans come from
numpy's default_rng, bulk tensors from a torch Generator on the target device.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

SEED_BASE = 251221450

# d, V, prompts, G, L_max, (len_lo, len_hi), W std, reward kind, eps_low, eps_high, beta, ent_coef
CONFIGS = {
    0: dict(name="tiny", d=256, V=4096, prompts=4, G=4, L_max=16, len_range=(16, 16), w_std=0.02,
            reward=("bernoulli", 0.5), eps=(0.2, 0.2), beta=0.04, ent_coef=0.0),
    1: dict(name="3b-head", d=2048, V=151936, prompts=8, G=8, L_max=512, len_range=(64, 512), w_std=0.02,
            reward=("bernoulli", 0.4), eps=(0.2, 0.2), beta=0.04, ent_coef=0.0),
    2: dict(name="7b-head", d=3584, V=152064, prompts=16, G=8, L_max=1024, len_range=(128, 1024), w_std=0.015,
            reward=("uniform", None), eps=(0.2, 0.2), beta=0.04, ent_coef=0.0),
    3: dict(name="long-agentic", d=2560, V=151936, prompts=4, G=8, L_max=4096, len_range=(4096, 4096), w_std=0.02,
            reward=("bernoulli", 0.3), eps=(0.2, 0.2), beta=0.04, ent_coef=0.0, span_mask=0.30),
    4: dict(name="large-batch-asym", d=2048, V=151936, prompts=64, G=16, L_max=512, len_range=(32, 512), w_std=0.02,
            reward=("bernoulli", 0.5), eps=(0.2, 0.28), beta=0.0, ent_coef=1e-3, zero_var_frac=0.25),
}


@dataclass
class Workload:
    cfg_id: int
    name: str
    d: int
    V: int
    G: int
    n_seq: int
    L_max: int
    T: int
    eps_low: float
    eps_high: float
    beta: float
    ent_coef: float
    H: torch.Tensor = None          # [T, d] bf16
    W: torch.Tensor = None          # [V, d] bf16
    tokens: torch.Tensor = None     # [T] int32
    mask: torch.Tensor = None       # [T] uint8
    seq_offsets: torch.Tensor = None  # [n_seq+1] int32 (row range of each response, padding included)
    rewards: torch.Tensor = None    # [n_seq] f32
    old_logp: torch.Tensor = None   # [T] f32
    ref_logp: torch.Tensor = None   # [T] f32 or None (beta == 0)
    n_valid: int = 0
    extra: dict = field(default_factory=dict)


def _lengths_and_mask(cfg, n_seq, L_max, rng):
    lo, hi = cfg["len_range"]
    if L_max != cfg["L_max"]:
        # shrunk parity case: keep the shape of the length distribution
        lo = max(1, lo * L_max // cfg["L_max"])
        hi = max(lo, hi * L_max // cfg["L_max"])
    lens = rng.integers(lo, hi + 1, size=n_seq)
    mask = np.zeros((n_seq, L_max), dtype=np.uint8)
    for i, n in enumerate(lens):
        mask[i, :n] = 1
    frac = cfg.get("span_mask")
    if frac:
        # multi-turn rollouts: observation / tool-output spans are excluded from the loss
        s_lo = max(2, 32 * L_max // cfg["L_max"])
        s_hi = max(s_lo + 1, 256 * L_max // cfg["L_max"])
        for i in range(n_seq):
            target = int(frac * lens[i])
            guard = 0
            while (lens[i] - mask[i].sum()) < target and guard < 10000:
                span = int(rng.integers(s_lo, s_hi + 1))
                start = int(rng.integers(1, max(2, lens[i] - span)))
                mask[i, start:start + span] = 0
                guard += 1
            mask[i, 0] = 1
    return lens, mask


def _rewards(cfg, n_seq, G, rng):
    kind, p = cfg["reward"]
    if kind == "uniform":
        r = rng.uniform(size=n_seq)
    else:
        r = (rng.uniform(size=n_seq) < p).astype(np.float64)
    zf = cfg.get("zero_var_frac", 0.0)
    if zf:
        for g in range(n_seq // G):
            if rng.uniform() < zf:
                r[g * G:(g + 1) * G] = float(rng.uniform() < 0.5)
    return r.astype(np.float32)


@torch.no_grad()
def sample_tokens_and_logp(H, W, rows, gen, chunk_rows=2048):
    """Rollout stand-in: y ~ softmax(H W^T) (Gumbel-max) and log softmax(.)[y] for the given rows."""
    dev = H.device
    y = torch.zeros(H.shape[0], dtype=torch.int32, device=dev)
    lp = torch.zeros(H.shape[0], dtype=torch.float32, device=dev)
    Wf = W.float()
    for s in range(0, rows.numel(), chunk_rows):
        idx = rows[s:s + chunk_rows]
        z = H[idx].float() @ Wf.T
        u = torch.rand(z.shape, generator=gen, device=dev, dtype=torch.float32).clamp_(1e-20, 1.0)
        tok = torch.argmax(z - torch.log(-torch.log(u)), dim=1)
        lse = torch.logsumexp(z, dim=1)
        lp[idx] = z.gather(1, tok[:, None])[:, 0] - lse
        y[idx] = tok.to(torch.int32)
    return y, lp


def make_workload(cfg_id, device=None, prompts=None, L_max=None, seed=None, sigma_old=0.05, sigma_ref=0.1,
                  peaked_frac=0.0, d=None, V=None):
    """Build workload `cfg_id`; `prompts` / `L_max` shrink it for oracle-sized parity cases."""
    cfg = CONFIGS[cfg_id]
    if device is None:
        device = torch.device("cuda" if torch.cuda.is_available() else "cpu")
    device = torch.device(device)
    seed = SEED_BASE + cfg_id if seed is None else seed
    rng = np.random.default_rng(seed)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    d = cfg["d"] if d is None else d
    V = cfg["V"] if V is None else V
    G = cfg["G"]
    n_prompts = cfg["prompts"] if prompts is None else prompts
    L = cfg["L_max"] if L_max is None else L_max
    n_seq = n_prompts * G
    T = n_seq * L
    lens, mask_np = _lengths_and_mask(cfg, n_seq, L, rng)
    rewards_np = _rewards(cfg, n_seq, G, rng)

    H = torch.randn(T, d, generator=gen, device=device, dtype=torch.float32)
    if peaked_frac > 0:
        sel = torch.rand(T, generator=gen, device=device) < peaked_frac
        H[sel] *= 40.0
    H = H.to(torch.bfloat16)
    W = (torch.randn(V, d, generator=gen, device=device, dtype=torch.float32) * cfg["w_std"]).to(torch.bfloat16)
    mask = torch.from_numpy(mask_np.reshape(-1)).to(device)
    rows = torch.nonzero(mask, as_tuple=False)[:, 0]
    tokens, base_lp = sample_tokens_and_logp(H, W, rows, gen)
    old = base_lp + sigma_old * torch.randn(T, generator=gen, device=device)
    ref = base_lp + sigma_ref * torch.randn(T, generator=gen, device=device)
    beta = cfg["beta"]
    w = Workload(cfg_id=cfg_id, name=cfg["name"], d=d, V=V, G=G, n_seq=n_seq, L_max=L, T=T,
                 eps_low=cfg["eps"][0], eps_high=cfg["eps"][1], beta=beta, ent_coef=cfg["ent_coef"])
    w.H, w.W, w.tokens, w.mask = H, W, tokens, mask
    w.seq_offsets = torch.arange(0, T + 1, L, dtype=torch.int32, device=device)
    w.rewards = torch.from_numpy(rewards_np).to(device)
    w.old_logp = old * mask
    w.ref_logp = (ref * mask) if beta != 0.0 else None
    w.n_valid = int(mask.sum().item())
    w.extra = dict(lens=lens, seed=seed)
    return w


def make_reference_model(w, d_ref=None, drift=0.05, seed_offset=7919):
    """Frozen reference model for the full-distribution KL: hidden states H_ref [T, d_ref] and LM head
    W_ref [V, d_ref] (bf16).  With d_ref equal to the policy's d the reference is the policy before
    training: the same tensors plus a relative Gaussian drift, the situation of an RL run that started
    from the reference checkpoint.  With another d_ref it is an unrelated random model of that width
    with the same logit scale."""
    dev = w.H.device
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.extra["seed"] + seed_offset)
    d_ref = w.d if d_ref is None else d_ref
    if d_ref == w.d:
        H_ref = (w.H.float() + drift * torch.randn(w.T, w.d, generator=gen, device=dev)).to(torch.bfloat16)
        W_ref = (w.W.float() * (1.0 + drift * torch.randn(w.V, w.d, generator=gen, device=dev))).to(torch.bfloat16)
    else:
        w_std = float(w.W.float().std().item()) * (w.d / d_ref) ** 0.5
        H_ref = torch.randn(w.T, d_ref, generator=gen, device=dev).to(torch.bfloat16)
        W_ref = (torch.randn(w.V, d_ref, generator=gen, device=dev) * w_std).to(torch.bfloat16)
    return H_ref, W_ref
