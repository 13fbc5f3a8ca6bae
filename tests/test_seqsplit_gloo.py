"""The gather-and-merge host logic of the sequence-split decode on two gloo ranks (CPU): every rank holds the oracle
cache of its token range, the partials cross the process group, and the merged result equals the oracle's merge of the
same shards on every rank."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import mixkvq_oracle as O
from paper_2512_19206_b200 import seqsplit
from paper_2512_19206_b200 import workloads as W

sys.path.insert(0, os.path.dirname(__file__))


def test_shard_ranges():
    assert seqsplit.shard_ranges(1000, 2, 128) == [(0, 384), (384, 1000)]
    assert seqsplit.shard_ranges(100, 2, 128) == [(0, 0), (0, 100)]            # too short to split: rank 0 stays empty
    r = seqsplit.shard_ranges(131072 + 77, 8, 128)
    assert r[0] == (0, 16384) and r[-1] == (7 * 16384, 131072 + 77)
    assert all(a[1] == b[0] for a, b in zip(r, r[1:])) and all(t0 % 128 == 0 for t0, _ in r)


def _shard_partials(w, rng_range, k, v, q, qd):
    """Oracle partials [B, Hq, 128], [B, Hq] of the token range for every stream."""
    t0, t1 = rng_range
    out = np.zeros((w.batch, w.n_q_heads, O.D))
    lse = np.zeros((w.batch, w.n_q_heads))
    for b in range(w.batch):
        for hk in range(w.n_kv_heads):
            st = O.OracleStream(g=w.g, R=w.residual_len, G=w.group_size, score_bits=w.score_bits, tau_bf16=w.tau_bf16,
                                tau_u4=w.tau_u4)
            hs = slice(hk * w.g, (hk + 1) * w.g)
            if t1 > t0:
                st.append_many(k[b, hk, t0:t1], v[b, hk, t0:t1], q[b, hs, t0:t1])
            out[b, hs], lse[b, hs] = st.attention_partial(qd[b, hs], W.softmax_scale())
    return out, lse


def _inputs(tokens):
    w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=2, tokens=tokens, **W.P27)
    k, v, q = [t.to(torch.float32).numpy() for t in W.tokens(w, 0, 0, tokens)]
    qd = W.decode_query(w, 0, 3).to(torch.float32).numpy()
    return w, k, v, q, qd


def _rank(rank, world, port, tokens, q_out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w, k, v, q, qd = _inputs(tokens)
    ranges = seqsplit.shard_ranges(tokens, world, w.residual_len)
    out, lse = _shard_partials(w, ranges[rank], k, v, q, qd)
    merged = seqsplit.split_attention(torch.from_numpy(out), torch.from_numpy(lse),
                                      lambda o, l: torch.from_numpy(O.merge_partials(o.numpy(), l.numpy())))
    q_out.put((rank, merged.numpy()))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("tokens", [700, 90])
def test_two_ranks_gather_and_merge(tokens):
    from paper_2512_19206_b200.replicas import free_port
    world, port = 2, free_port()
    ctx = mp.get_context("spawn")
    q_out = ctx.Queue()
    procs = [ctx.Process(target=_rank, args=(r, world, port, tokens, q_out)) for r in range(world)]
    for p in procs:
        p.start()
    got = dict(q_out.get(timeout=240) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # the expected value: the oracle's merge of the same shards, computed here without any process group
    w, k, v, q, qd = _inputs(tokens)
    ranges = seqsplit.shard_ranges(tokens, world, w.residual_len)
    parts = [_shard_partials(w, r, k, v, q, qd) for r in ranges]
    want = O.merge_partials([p[0] for p in parts], [p[1] for p in parts])
    for r in range(world):
        assert np.array_equal(got[r], want)
