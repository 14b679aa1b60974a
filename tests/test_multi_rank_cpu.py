"""The N > 1 path on CPU: two gloo ranks, one shard of the sequence batch each.

Sequences are independent (own bandit state, Philox streams keyed by the global sequence id), so the path
shards by sequence with no collective on the data path; the only cross-rank step is the bookkeeping of the
benchmark (rows summed, time taken as the maximum).  Checked here: (1) that bookkeeping, through the very
function bench.py uses; (2) that two shards, each told the global ids of its sequences, reproduce the
full-batch run decision by decision (with the CPU oracle standing in for the device: the sharding rule
is the same, global id = seq_offset + local index)."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2511_02017_b200 import synth_inputs as si  # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _run_rounds(w, seq_ids, rounds):
    """Oracle rounds over the sequences `seq_ids` of workload w; returns (tokens, accept_len, next_token, cnt)."""
    from tests.lockstep import make_oracle
    ora = make_oracle(w, seq_ids)
    K = w.k_max
    outs = []
    for rnd in range(rounds):
        d, t = si.round_logits(w, rnd, "cpu")
        Dn, Tn = si.to_numpy_bits(d[seq_ids]), si.to_numpy_bits(t[seq_ids])
        toks = np.full((len(seq_ids), K), -1, np.int32)
        for i in range(K):
            toks[:, i] = ora.draft_step(Dn[:, i, :])["token"]
        v = ora.verify(Dn, Tn, toks)
        ora.update()
        outs.append((toks.copy(), v["accept_len"].copy(), v["next_token"].copy()))
    return outs, ora.view("cnt").copy()


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        # (1) bookkeeping: rows add up, the slowest rank sets the time
        rows, ms = bench.aggregate(1000 + rank, 5.0 + 2.0 * rank, world, True)
        assert rows == sum(1000 + r for r in range(world)), rows
        assert ms == 5.0 + 2.0 * (world - 1), ms
        # (2) this rank's shard of the batch
        w = si.Workload("shard", 6, 1032, "bf16", 4, 1, 5, "ts", "seq", seed=77, sigma="per_seq:0.2:1.5")
        per = w.n_seq // world
        ids = np.arange(rank * per, (rank + 1) * per)
        outs, cnt = _run_rounds(w, ids, 5)
        gathered = [None] * world
        dist.all_gather_object(gathered, (outs, cnt))
        if rank == 0:
            full, cnt_full = _run_rounds(w, np.arange(w.n_seq), 5)
            for rnd in range(5):
                for j in range(3):
                    cat = np.concatenate([g[0][rnd][j] for g in gathered])
                    assert np.array_equal(cat, full[rnd][j]), (rnd, j)
            assert np.array_equal(np.concatenate([g[1] for g in gathered]), cnt_full)
        q.put((rank, "ok"))
    except Exception as e:  # noqa: BLE001
        q.put((rank, "failed: %r" % (e,)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_by_sequence():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=240) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
    assert res == {0: "ok", 1: "ok"}, res
