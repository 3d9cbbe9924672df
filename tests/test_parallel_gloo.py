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
    par.allreduce_gradients(dW, loss)
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
