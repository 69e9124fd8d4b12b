"""Multi-rank host logic on CPU: two gloo ranks shard the tokens, code their shares (with the CPU oracle standing
in for the device codec), exchange payload bytes, and the concatenation equals the single-process payload."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_04991_b200 import shard, synth


def test_ranges_partition_the_tokens():
    for T in (0, 1, 7, 128, 131072, 131073):
        for world in (1, 2, 3, 8):
            r = shard.all_ranges(T, world)
            assert r[0][0] == 0 and r[-1][1] == T
            assert all(a[1] == b[0] for a, b in zip(r, r[1:]))
            sizes = [b - a for a, b in r]
            assert max(sizes) - min(sizes) <= 1
    assert shard.payload_range(2208, 10, 12) == (22080, 26496)
    with pytest.raises(ValueError):
        shard.token_range(10, 2, 2)


def _worker(rank, world, port, T, d, g, bits, k, out_dir):
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    gen = synth.generator(123)
    X = synth.activations(T, d, synth.channel_scale(d, 9), gen)      # same draw on every rank
    R = synth.affine_noisy_reference(X, g, gen)
    step = np.full((2, d), 0.02, np.float32)
    inv = (np.float32(1) / step).astype(np.float32)
    rec = oracle.record_bytes(d, g, bits, k)
    # the function the benchmark's strong-scaling mode uses: code the own token range into the own byte range of a
    # full-length buffer, then exchange the byte ranges
    payload = torch.zeros(T * rec, dtype=torch.uint8)

    def encode_range(a, b):
        mine = oracle.encode(d, g, bits, k, synth.bf16_bits(X[a:b]), ref_base=synth.bf16_bits(R[a:b]), step=step, inv_step=inv)
        lo, hi = shard.payload_range(rec, a, b)
        assert mine.size == hi - lo
        payload[lo:hi] = torch.from_numpy(mine)

    a, b = shard.sharded_encode(encode_range, T, rec, payload, rank, world)
    assert (a, b) == shard.token_range(T, rank, world)
    full = payload.numpy()
    # max-over-ranks reduction as the benchmark does for its timing
    t = torch.tensor([float(rank + 1)])
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    assert t.item() == world
    if rank == 0:
        np.save(os.path.join(out_dir, "full.npy"), full)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_reassemble_the_payload(tmp_path, orc):
    T, d, g, bits, k = 37, 256, 64, 4, 4
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(2, port, T, d, g, bits, k, str(tmp_path)), nprocs=2, join=True)
    full = np.load(tmp_path / "full.npy")
    gen = synth.generator(123)
    X = synth.activations(T, d, synth.channel_scale(d, 9), gen)
    R = synth.affine_noisy_reference(X, g, gen)
    step = np.full((2, d), 0.02, np.float32)
    inv = (np.float32(1) / step).astype(np.float32)
    want = orc.encode(d, g, bits, k, synth.bf16_bits(X), ref_base=synth.bf16_bits(R), step=step, inv_step=inv)
    assert np.array_equal(full, want)
