"""Two CPU ranks (gloo): sharding tokens across ranks needs no collective on the data path.

Each rank encodes and multiplies only its own rows (CPU oracle standing in for a GPU's kernels);
gathering the shards reproduces the single-process result bit for bit.
"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import gen
import oracle
from paper_2512_05409_b200 import row_shard


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, M, N, K, b, k, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        X = gen.bf16_bits(gen.activations(M, K, seed=5))
        W = gen.bf16_bits(gen.weights(N, K, seed=5))
        lo, hi = row_shard(M, world, rank)
        enc = oracle.encode(b, k, X[lo:hi])
        pw = oracle.pack_weights(b, k, W)
        acc, _, out = oracle.gemm(b, k, enc, pw)
        # gather the shards on every rank (the only communication; not part of the path)
        pieces = [None] * world
        dist.all_gather_object(pieces, (lo, hi, enc.dq4, enc.vals, enc.idx, enc.shift, acc, out))
        if rank == 0:
            q.put(pieces)
    finally:
        dist.destroy_process_group()


def test_row_shard_partitions():
    for M in (0, 1, 7, 64, 4097):
        for w in (1, 2, 3, 8):
            ranges = [row_shard(M, w, r) for r in range(w)]
            assert ranges[0][0] == 0 and ranges[-1][1] == M
            assert all(a[1] == b_[0] for a, b_ in zip(ranges, ranges[1:]))
            sizes = [hi - lo for lo, hi in ranges]
            assert max(sizes) - min(sizes) <= 1


def test_two_ranks_reproduce_the_single_process_result():
    M, N, K, b, k, world = 37, 24, 256, 64, 8, 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, M, N, K, b, k, q)) for r in range(world)]
    for p in procs:
        p.start()
    pieces = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    X = gen.bf16_bits(gen.activations(M, K, seed=5))
    W = gen.bf16_bits(gen.weights(N, K, seed=5))
    enc = oracle.encode(b, k, X)
    acc, _, out = oracle.gemm(b, k, enc, oracle.pack_weights(b, k, W))
    pieces.sort(key=lambda t: t[0])
    assert pieces[0][0] == 0 and pieces[-1][1] == M
    assert np.array_equal(np.concatenate([p[2] for p in pieces]), enc.dq4)
    assert np.array_equal(np.concatenate([p[3] for p in pieces]), enc.vals)
    assert np.array_equal(np.concatenate([p[4] for p in pieces]), enc.idx)
    assert np.array_equal(np.concatenate([p[5] for p in pieces]), enc.shift)
    assert np.array_equal(np.concatenate([p[6] for p in pieces]), acc)
    assert np.array_equal(np.concatenate([p[7] for p in pieces]), out)
