"""The ID-partitioned exchange (paper, Section 3: requests are served "by partition of Image ID") on CPU tensors:
routing of IDs to their owners, rows back to the requesters in the order of their ID lists, gradient rows to the owners
sender by sender in row order.  The in-process form (all ranks in one process) is checked against the definition; the
torch.distributed form is run as two gloo ranks and must move exactly what the in-process form moves."""
import os
import socket
import subprocess
import sys
import textwrap

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _ids(seed, n, vocab):
    rng = np.random.default_rng(seed)
    ids = rng.integers(0, vocab, n).astype(np.int32)
    if n > 3:
        ids[1] = ids[2]                                    # a repeat
    return torch.from_numpy(ids)


def test_loopback_exchange_follows_the_partition_rule():
    from paper_1806_03925_b200.sharded import LoopbackExchange, partition_by_owner, shard_rows
    W, V, dim = 3, 1000, 4
    table = torch.arange(V * dim, dtype=torch.float32).reshape(V, dim)
    shards = [table[r::W] for r in range(W)]
    assert [s.shape[0] for s in shards] == [shard_rows(V, r, W) for r in range(W)]
    ids = [_ids(10 + s, n, V) for s, n in enumerate((17, 0, 5))]           # uneven, one rank asks for nothing
    ex = LoopbackExchange(W)
    routes = ex.route(ids)
    for o, rt in enumerate(routes):
        # what arrives at owner o: sender by sender, each sender's entries for o in its own order, as owner-local rows
        want = torch.cat([(i[i % W == o] // W) for i in ids]).to(torch.int32)
        assert torch.equal(rt.recv_local, want)
        assert rt.recv_counts == [int((i % W == o).sum()) for i in ids]
        assert sum(rt.send_counts) == len(ids[o])
    # rows back: every requester gets the table rows of its IDs, in the order of its ID list
    got = ex.reply(routes, [shards[o][rt.recv_local.long()] for o, rt in enumerate(routes)])
    for s in range(W):
        assert torch.equal(got[s], table[ids[s].long()])
    # gradient rows out: row k of sender s carries (s, k); the owner sees them aligned with recv_local
    rows = [torch.stack([torch.full((len(i),), float(s)), torch.arange(len(i), dtype=torch.float32)], 1) for s, i in enumerate(ids)]
    at_owner = ex.push(routes, rows)
    for o in range(W):
        want = torch.cat([rows[s][ids[s] % W == o] for s in range(W)])
        assert torch.equal(at_owner[o], want)
    # a negative ID is routed somewhere and stays negative there (its owner refuses it)
    order, counts, local = partition_by_owner(torch.tensor([-5, 7], dtype=torch.int32), W)
    assert int(local[0]) < 0 and sum(counts) == 2


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_move_what_the_in_process_exchange_moves(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(textwrap.dedent("""
        import os, sys
        import numpy as np, torch, torch.distributed as dist
        from paper_1806_03925_b200.sharded import DistExchange, LoopbackExchange
        rank, W = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
        dist.init_process_group("gloo", rank=rank, world_size=W)
        V, dim = 501, 3
        table = torch.arange(V * dim, dtype=torch.float32).reshape(V, dim)
        def ids_of(s):
            rng = np.random.default_rng(100 + s)
            return torch.from_numpy(rng.integers(0, V, 40 + 13 * s).astype(np.int32))
        all_ids = [ids_of(s) for s in range(W)]
        rows_of = lambda s: torch.stack([torch.full((len(all_ids[s]),), float(s)), torch.arange(len(all_ids[s]), dtype=torch.float32)], 1)
        # every rank can work out the whole exchange in process ...
        lb = LoopbackExchange(W)
        lr = lb.route(all_ids)
        l_reply = lb.reply(lr, [table[o::W][r.recv_local.long()] for o, r in enumerate(lr)])
        l_push = lb.push(lr, [rows_of(s) for s in range(W)])
        # ... and takes part in the real one with its own share only
        ex = DistExchange(rank, W)
        (rt,) = ex.route([all_ids[rank]])
        assert torch.equal(rt.recv_local, lr[rank].recv_local) and rt.recv_counts == lr[rank].recv_counts
        (got,) = ex.reply([rt], [table[rank::W][rt.recv_local.long()]])
        assert torch.equal(got, l_reply[rank]) and torch.equal(got, table[all_ids[rank].long()])
        (arrived,) = ex.push([rt], [rows_of(rank)])
        assert torch.equal(arrived, l_push[rank])
        dist.barrier()
        open(sys.argv[1] + "/ok%d" % rank, "w").write("ok")
        dist.destroy_process_group()
    """))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), str(script), str(tmp_path)]
    out = subprocess.run(cmd, cwd=ROOT, env=dict(os.environ, PYTHONPATH=ROOT, OMP_NUM_THREADS="1"), capture_output=True,
                         text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-3000:]
    assert os.path.exists(tmp_path / "ok0") and os.path.exists(tmp_path / "ok1")
