"""World-size-2 check (gloo, CPU) of the data-parallel plumbing: sharding by whole prompts, the
global token-mean weight and the gradient all-reduce reproduce the single-process result.  The
float64 oracle stands in for the per-rank compute."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import grpo_oracle as O


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _problem():
    rng = np.random.default_rng(3)
    prompts, G, L, d, V = 3, 4, 6, 8, 24
    T = prompts * G * L
    H = rng.normal(size=(T, d))
    W = rng.normal(size=(V, d)) * 0.4
    tok = rng.integers(0, V, size=T)
    mask = (rng.uniform(size=T) < 0.8).astype(np.uint8)
    lp, _, _ = O.token_logprobs(H, W, tok)
    old = lp + rng.normal(size=T) * 0.3
    ref = lp + rng.normal(size=T) * 0.2
    rewards = (rng.uniform(size=prompts * G) < 0.5).astype(np.float64)
    return dict(prompts=prompts, G=G, L=L, H=H, W=W, tok=tok, mask=mask, old=old, ref=ref, rewards=rewards)


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2512_21450_b200 import parallel as par
    P = _problem()
    start, count = par.shard_prompts(P["prompts"], world, rank)
    rows = slice(start * P["G"] * P["L"], (start + count) * P["G"] * P["L"])
    seqs = slice(start * P["G"], (start + count) * P["G"])
    mask = torch.from_numpy(P["mask"][rows])
    tw = par.global_token_weight(mask)
    adv_seq = O.grpo_advantages(P["rewards"][seqs], P["G"])            # groups are whole on a rank
    n_rows = rows.stop - rows.start
    adv = O.broadcast_to_tokens(adv_seq, np.arange(0, n_rows + 1, P["L"]), n_rows)
    out = O.policy_loss_fwd_bwd(P["H"][rows], P["W"], P["tok"][rows], P["old"][rows], P["ref"][rows], adv,
                                P["mask"][rows], 0.2, 0.28, 0.04, ent_coef=0.01, token_weight=tw.double().numpy())
    dW = torch.from_numpy(out["dW"].copy())
    loss = torch.tensor([out["loss"]], dtype=torch.float64)
    # the same gradient handed over slab by slab, as the backward pass reports it (7 vocabulary rows per
    # slab here, ragged last slab): must give the same sum as one all-reduce of the whole matrix
    dW_slabs = torch.from_numpy(out["dW"].copy())
    loss_slabs = loss.clone()
    red = par.SlabGradientReducer(dW_slabs)
    red.begin()
    V = dW.shape[0]
    for k, r0 in enumerate(range(0, V, 7)):
        red.on_slab(k, r0, min(V, r0 + 7))
    red.finish(loss_slabs)
    assert [s[1] for s in red.slabs] == list(range(0, V, 7)) and red.slabs[-1][2] == V
    par.allreduce_gradients(dW, loss)
    assert torch.equal(dW, dW_slabs) and torch.equal(loss, loss_slabs)
    if rank == 0:
        q.put((dW.numpy(), float(loss.item()), int(par.global_valid_count(mask).item())))
    else:
        par.global_valid_count(mask)
    dist.barrier()
    dist.destroy_process_group()


def test_shard_prompts_partition():
    from paper_2512_21450_b200 import parallel as par
    for n in (1, 3, 8, 64):
        for world in (1, 2, 3, 8):
            blocks = [par.shard_prompts(n, world, r) for r in range(world)]
            assert sum(c for _, c in blocks) == n
            pos = 0
            for s, c in blocks:
                assert s == pos
                pos += c
            assert max(c for _, c in blocks) - min(c for _, c in blocks) <= 1


def test_two_rank_data_parallel_matches_single_process():
    world = 2
    port = _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    dW, loss, n_global = q.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    P = _problem()
    T = P["H"].shape[0]
    adv = O.broadcast_to_tokens(O.grpo_advantages(P["rewards"], P["G"]), np.arange(0, T + 1, P["L"]), T)
    ref = O.policy_loss_fwd_bwd(P["H"], P["W"], P["tok"], P["old"], P["ref"], adv, P["mask"], 0.2, 0.28, 0.04,
                                ent_coef=0.01)
    assert n_global == int(P["mask"].sum())
    # weights travel as fp32 (1/N rounded), hence the 1e-6 relative tolerance
    assert abs(loss - ref["loss"]) <= 1e-6 * abs(ref["loss"])
    assert np.abs(dW - ref["dW"]).max() <= 1e-6 * np.abs(ref["dW"]).max()


# ----------------------------------------------------------------------------- vocabulary-parallel head
class _OracleCompute:
    """Stands in for the GPU context on CPU ranks: the three per-rank calls, from the float64 oracle."""

    def rl_shard_logit_stats(self, H, W_shard, tokens, mask, vocab_offset, V_total):
        return torch.from_numpy(O.shard_logit_stats(H.numpy(), W_shard.numpy(), tokens.numpy(), vocab_offset, mask.numpy()))

    def rl_merge_logit_stats(self, stats, mask):
        return tuple(torch.from_numpy(x) for x in O.merge_logit_stats(stats.numpy(), mask.numpy()))

    def rl_policy_loss_shard_bwd(self, H, W_shard, tokens, old, ref, adv, mask, vocab_offset, V_total, logp, ent, lse,
                                 eps_low, eps_high, beta, **kw):
        o = O.policy_loss_shard_bwd(H.numpy(), W_shard.numpy(), tokens.numpy(), vocab_offset, logp.numpy(), ent.numpy(),
                                    lse.numpy(), old.numpy(), ref.numpy(), adv.numpy(), mask.numpy(), eps_low, eps_high,
                                    beta, **kw)
        return dict(loss=torch.tensor([o["loss"]], dtype=torch.float64), dH=torch.from_numpy(o["dH_partial"]), dW=torch.from_numpy(o["dW_shard"]))


def _vocab_worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2512_21450_b200 import parallel as par
    P = _problem()
    V = P["W"].shape[0]
    off, size = par.shard_vocab(V, world, rank, multiple=8)
    T = P["H"].shape[0]
    adv = O.broadcast_to_tokens(O.grpo_advantages(P["rewards"], P["G"]), np.arange(0, T + 1, P["L"]), T)
    t = torch.from_numpy
    out = par.vocab_parallel_loss_fwd_bwd(_OracleCompute(), t(P["H"]), t(P["W"][off:off + size].copy()), t(P["tok"]),
                                          t(P["old"]), t(P["ref"]), t(adv), t(P["mask"]), off, V, 0.2, 0.28, 0.04,
                                          ent_coef=0.01)
    q.put((rank, off, size, out["dW"].numpy(), out["dH"].numpy(), float(out["loss"].item()), out["logp"].numpy()))
    dist.barrier()
    dist.destroy_process_group()


def test_shard_vocab_partition():
    from paper_2512_21450_b200 import parallel as par
    for V in (1, 255, 256, 4096, 151936, 152064):
        for world in (1, 2, 3, 8):
            pos = 0
            for r in range(world):
                off, size = par.shard_vocab(V, world, r)
                assert off == pos and size >= 0 and (off % 256 == 0 or size == 0)
                pos += size
            assert pos == V


def test_two_rank_vocab_parallel_matches_single_process():
    world = 2
    port = _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_vocab_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted([q.get(timeout=120) for _ in range(world)], key=lambda x: x[0])
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    P = _problem()
    T = P["H"].shape[0]
    adv = O.broadcast_to_tokens(O.grpo_advantages(P["rewards"], P["G"]), np.arange(0, T + 1, P["L"]), T)
    ref = O.policy_loss_fwd_bwd(P["H"], P["W"], P["tok"], P["old"], P["ref"], adv, P["mask"], 0.2, 0.28, 0.04,
                                ent_coef=0.01)
    assert got[0][1] == 0 and got[0][2] > 0 and got[1][1] == got[0][2] and got[1][1] + got[1][2] == P["W"].shape[0]
    for rank, off, size, dW, dH, loss, logp in got:
        assert abs(loss - ref["loss"]) <= 1e-13 * max(1.0, abs(ref["loss"]))
        assert np.abs(logp - ref["logp"]).max() <= 1e-12
        assert np.abs(dW - ref["dW"][off:off + size]).max() <= 1e-13
        assert np.abs(dH - ref["dH"]).max() <= 1e-13          # summed over the two ranks
