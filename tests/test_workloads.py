"""The seeded input generators and the multi-rank plumbing of the benchmark (CPU only)."""
import math
import os
import socket
import sys

import numpy as np
import torch
import torch.multiprocessing as mp

import oracle
from paper_2607_21599_b200 import workloads as W


def test_generator_is_deterministic_and_counter_based():
    a = W.normal_bf16((1000, 4, 8), 1234)
    b = W.normal_bf16((1000, 4, 8), 1234)
    assert torch.equal(a, b)
    assert not torch.equal(a, W.normal_bf16((1000, 4, 8), 1235))
    # element i depends on (seed, i) only: a longer draw starts with the shorter one
    long = W.standard_normal(5000, 77)
    assert torch.equal(long[:100], W.standard_normal(100, 77))
    x = W.standard_normal(200000, 5).numpy()
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01
    u = W.uniform01(100000, 9).numpy()
    assert 0.0 <= u.min() and u.max() < 1.0 and abs(u.mean() - 0.5) < 0.01
    # the tensor form and the integer form of the hash agree
    c = torch.arange(0, 5, dtype=torch.int64)
    t = W.splitmix64_tensor(c, 42).tolist()
    assert [v & ((1 << 64) - 1) for v in t] == [W.splitmix64_int(42 + i) for i in range(5)]


def test_layers_and_tensors_are_independent():
    w = W.tiny(num_important=oracle.num_important)
    a, b = W.make_layer(w, 0), W.make_layer(w, 1)
    assert not torch.equal(a["q_fresh"], b["q_fresh"])
    assert not torch.equal(a["k_fresh"][: w.L_d], a["k_cached"])
    assert a["scores"].shape == (w.n_sig, w.L_d) and a["scores"].dtype == torch.float32
    assert a["q_fresh"].shape == (w.N, w.n_q_heads, w.head_dim)


def test_workload_sizes_match_the_stated_configurations():
    c = W.CONFIGS
    assert (c["c0"].k, c["c1"].k, c["c2"].k, c["c3"].k) == (154, 922, 1639, 6554)
    # the stated counts are what the oracle's and the library's counting rules give
    from paper_2607_21599_b200 import api, build
    build.build()
    for w in list(c.values()) + list(W.EXTRA_CONFIGS.values()):
        assert w.k == oracle.num_important(w.L_d, w.r) == api.daf_num_important(w.L_d, w.r), w.name
    assert c["c0"].n_docs == 4 and c["c1"].n_docs == 12 and c["c2"].n_docs == 32 and c["c3"].n_docs == 64
    idx = W.given_indices(c["c0"])
    assert len(idx) == 154 and torch.all(idx[1:] > idx[:-1]) and 0 <= int(idx[0]) and int(idx[-1]) < 1024
    pts = W.sweep_points(oracle.num_important)
    assert len(pts) == 16 and {p.L_d for p in pts} == {2048, 8192, 16384, 32768}
    assert {p.name: p.k for p in pts}["c4_L32768_r0.30"] == 9831


def test_selection_share_of_hot_documents():
    """The clustered workload puts roughly 70 % of the selected tokens into 20 % of the documents."""
    w = W.CONFIGS["c3"]
    S = W.importance_scores(w, 0)
    idx = oracle.select(S.numpy(), w.k)
    per_doc = np.bincount(idx // w.doc_len, minlength=w.n_docs)
    top = np.sort(per_doc)[::-1][: math.ceil(0.2 * w.n_docs)].sum() / w.k
    assert 0.6 <= top <= 0.8, top


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, root):
    sys.path.insert(0, root)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.tiny(L_d=32, doc_len=8, L_q=3, num_important=oracle.num_important)
        layers = bench.replica_layers(rank, w)
        mine = W.make_layer(w, layers[0])["q_fresh"].float().sum().reshape(1).double()
        sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(sums, mine)
        assert len({float(x) for x in sums}) == world, "ranks generated the same replica"
        ids = [torch.zeros(len(layers), dtype=torch.int64) for _ in range(world)]
        dist.all_gather(ids, torch.tensor(layers, dtype=torch.int64))
        flat = torch.cat(ids).tolist()
        assert len(set(flat)) == len(flat), "layer seeds overlap between ranks"
        # durations are reported as the maximum over ranks
        assert bench.max_over_ranks(dist, float(rank + 1), "cpu") == float(world)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_distinct_replicas_and_report_the_slowest(repo_root):
    mp.spawn(_rank_main, args=(2, _free_port(), repo_root), nprocs=2, join=True)
