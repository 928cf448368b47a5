"""The multi-client exchange (Algorithm 1: gather of the messages, average of the decoded
updates) with two gloo ranks on CPU: the collective and slot layout are the product's, the
messages and the expected aggregate are the oracle's."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

N, P, WORLD = 50000, 0.01, 2


def _client_update(rank):
    from paper_1805_08768_b200 import workloads
    return workloads.normal_flat(N, 1e-3, 900 + rank)


def _worker(rank, world, port, out_dir):
    import oracle
    from paper_1805_08768_b200.exchange import StreamExchange
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ex = StreamExchange(oracle.stream_bytes(N, P), torch.device("cpu"))
        assert (ex.world, ex.rank) == (world, rank) and ex.capacity % 16 == 0
        stream, _ = oracle.encode(_client_update(rank), np.zeros(N, dtype=np.float32), P)
        ex.send[: stream.size] = torch.from_numpy(stream)
        ex.gather()
        weights = np.zeros(N, dtype=np.float32)
        got = []
        for r, slot in enumerate(ex.slots):
            hdr = oracle.parse_header(slot.numpy())
            got.append(slot.numpy()[: oracle.container_bytes(hdr.k, hdr.nbits)].copy())
        oracle.decode_apply(got, 1.0 / world, weights)
        np.save(os.path.join(out_dir, f"w{rank}.npy"), weights)
        np.save(os.path.join(out_dir, f"s{rank}.npy"), np.concatenate(got))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_gather_each_other_s_messages_and_agree(tmp_path):
    import oracle
    mp.spawn(_worker, args=(WORLD, 29621, str(tmp_path)), nprocs=WORLD, join=True)
    streams = [oracle.encode(_client_update(r), np.zeros(N, dtype=np.float32), P)[0] for r in range(WORLD)]
    want = np.zeros(N, dtype=np.float32)
    oracle.decode_apply(streams, 1.0 / WORLD, want)
    assert np.count_nonzero(want) >= oracle.kept_count(N, P)
    for r in range(WORLD):
        assert np.array_equal(np.load(tmp_path / f"s{r}.npy"), np.concatenate(streams))   # rank order
        assert np.array_equal(np.load(tmp_path / f"w{r}.npy").view(np.uint32), want.view(np.uint32))
