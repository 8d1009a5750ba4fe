"""world_size-2 gloo test of the multi-process plumbing used by bench.py --gpus N."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close()
    return p


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_1806_04090_b200 import dist as d
    r, lr, w = d.init("gloo")
    d.barrier()
    t_max = d.max_over_ranks(10.0 + 5.0 * rank)        # slowest rank decides the step time
    units = d.sum_over_ranks(100.0 * (rank + 1))       # whole-job units
    parts = d.shard_units([9.0, 1.0, 8.0, 2.0, 7.0], w)
    # exchange step: every rank's fixed-capacity payload buffer reaches every rank, in rank order
    import torch
    mine = (torch.arange(1000, dtype=torch.int64) * (rank + 3) % 251).to(torch.uint8)
    got = d.all_gather_bytes(mine)
    gathered_ok = len(got) == world and all(
        torch.equal(got[k], (torch.arange(1000, dtype=torch.int64) * (k + 3) % 251).to(torch.uint8)) for k in range(world))
    # the same exchange through the peer-buffer object (on CPU it falls back to the all-gather)
    peers = d.PeerPayloads(1000, torch.device("cpu"))
    peers.buf.copy_(mine)
    peers.publish()
    views = peers.views()
    gathered_ok = gathered_ok and len(views) == world and all(
        torch.equal(views[k], (torch.arange(1000, dtype=torch.int64) * (k + 3) % 251).to(torch.uint8)) for k in range(world))
    peers.release()
    d.barrier()
    d.finish()
    q.put((r, w, t_max, units, parts, gathered_ok))


def test_two_rank_reduction_and_sharding():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[0] for r in res] == [0, 1]
    for r in res:
        assert r[1] == 2 and r[2] == 15.0 and r[3] == 300.0
        assert r[4] == [[0, 3, 4], [1, 2]] or sorted(sum(r[4], [])) == [0, 1, 2, 3, 4]
        assert r[5]
    assert res[0][4] == res[1][4]                      # same partition on every rank


def test_single_process_defaults():
    from paper_1806_04090_b200 import dist as d
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert d.env_world() == (0, 0, 1)
    assert d.max_over_ranks(3.5) == 3.5 and d.sum_over_ranks(2.0) == 2.0
    assert d.shard_units([1, 2, 3], 1) == [[0, 1, 2]]
    import torch
    buf = torch.arange(16, dtype=torch.uint8)
    assert len(d.all_gather_bytes(buf)) == 1 and d.all_gather_bytes(buf)[0] is buf
