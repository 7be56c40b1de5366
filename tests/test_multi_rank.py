"""The N > 1 path on CPU: two gloo ranks shard the token rows, each encodes its own range (with the
oracle standing in for the GPU here), and the job-level figures are reduced the way bench.py does."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import tsq_ref as R
from paper_2511_04002_b200 import shard, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_token_ranges_partition_the_rows():
    for tokens in (0, 1, 7, 64, 8192, 8193):
        for world in (1, 2, 3, 8):
            spans = [shard.token_range(tokens, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == tokens
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard.token_range(8, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.c1_prefill()
        raw = synth.raw_u16(synth.make(w))
        a, b = shard.token_range(raw.shape[0], rank, world)
        blob = R.encode(raw[a:b], R.F16, w.tau, list(w.bits), w.delta)       # this rank's own blob
        np.save(os.path.join(out_dir, "y%d.npy" % rank), R.decode(blob))
        np.save(os.path.join(out_dir, "bits%d.npy" % rank), R.sections(blob)["bits"])
        ms, nbytes, launches = shard.reduce_job(10.0 + rank, 1000.0 * (rank + 1), 3 + rank, "cpu")
        assert (ms, nbytes, launches) == (10.0 + world - 1, 1000.0 * world * (world + 1) / 2, 3 * world + 1)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_without_a_data_collective(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    w = synth.c1_prefill()
    raw = synth.raw_u16(synth.make(w))
    whole = R.encode(raw, R.F16, w.tau, list(w.bits), w.delta)
    y = np.concatenate([np.load(tmp_path / ("y%d.npy" % r)) for r in range(world)])
    bits = np.concatenate([np.load(tmp_path / ("bits%d.npy" % r)) for r in range(world)])
    # rows are independent: the shards' reconstructions and bit-widths are those of the unsharded call
    assert np.array_equal(y, R.decode(whole))
    assert np.array_equal(bits, R.sections(whole)["bits"])


def test_reduce_job_without_a_process_group():
    assert shard.reduce_job(1.5, 10, 2, "cpu") == (1.5, 10.0, 2)


def test_bench_launches_its_own_ranks(capfd):
    """`bench.py --gpus N` started plainly launches N ranks under torch.distributed.run on 127.0.0.1.  Here, without a
    GPU, the launcher is driven with the CPU arm: rank 0 prints the one JSON line, the other rank exits 0."""
    import importlib.util
    import json
    spec = importlib.util.spec_from_file_location("bench_for_test", os.path.join(ROOT, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    rc = bench.launch_ranks(2, ["--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "3", "--workload", "c1"])
    assert rc == 0
    out = capfd.readouterr().out
    lines = [json.loads(l) for l in out.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2
    assert lines[0]["config"]["workload"].startswith("c1_") and "sample" in lines[0]
