"""Token-sharded driver (paper_2602_23111_b200/sharded.py) as two gloo ranks on CPU.  The driver is
plumbing over a basis object; here the basis is a stand-in built on the CPU oracle, so that the
collective logic (what is summed, what stays local, that every rank ends with the same U, Q and
the full-batch gradient) is checked without a GPU."""
import json
import os
import subprocess
import sys
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, {root!r})
    import numpy as np
    import torch
    import torch.distributed as dist
    from oracle import prac_oracle as orc
    from paper_2602_23111_b200.sharded import ShardedCompressor, shard_rows

    class OracleBasis:
        # the calls ShardedCompressor makes, on float64 CPU tensors through the oracle's definitions
        def __init__(self, d, k, r):
            self.d, self.k, self.r = d, k, r
        def gram(self, X, ws=None):
            return X.T @ X
        def fit_principal_gram(self, C, seed=0, draw_counter=0, ws=None):
            w, V = np.linalg.eigh(C.numpy())
            self.U = V[:, ::-1][:, :self.k].copy()
        def draw_random(self, seed=0, draw_counter=0, ws=None):
            self.Q = orc.random_basis(self.U, orc.gaussian_draw(seed, draw_counter, self.d, self.r))
            self.c = orc.scale_factor(self.d, self.k, self.r)
        def compress(self, X, out=None):
            return torch.from_numpy(orc.compress(X.numpy(), self.U, self.Q))
        def weight_grad_partial(self, dY, Z, ws=None):
            return dY.T @ Z
        def weight_grad_finish(self, M, out=None):
            P = np.concatenate([self.U, self.c * self.Q], axis=1)
            return torch.from_numpy(M.numpy() @ P.T)

    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    N, d, k, r, d_out = 61, 12, 3, 4, 5
    rng = np.random.default_rng(7)
    X = rng.standard_normal((N, d)) * np.linspace(3.0, 0.3, d)
    dY = rng.standard_normal((N, d_out))
    b0, b1 = shard_rows(N, world, rank)
    sc = ShardedCompressor(OracleBasis(d, k, r))
    sc.fit(torch.from_numpy(X[b0:b1]), seed=11, draw_counter=2)
    Z = sc.compress(torch.from_numpy(X[b0:b1]))
    dW = sc.weight_grad(torch.from_numpy(dY[b0:b1]), Z)
    # full-batch answers from the oracle alone
    U0, Q0, c0 = orc.fit_basis(X, k, r, seed=11, draw_counter=2)
    dW0 = orc.weight_grad(dY, orc.compress(X, U0, Q0), U0, Q0, c0)
    out = {{"rank": rank, "rows": [b0, b1],
           "proj_u": orc.projector_distance(sc.basis.U, U0), "proj_q": orc.projector_distance(sc.basis.Q, Q0),
           "dw_err": orc.rel_fro(dW.numpy(), dW0), "bytes": sc.bytes_reduced,
           "u_sum": float(np.abs(sc.basis.U).sum()), "q_sum": float(np.abs(sc.basis.Q).sum())}}
    print(json.dumps(out))
    dist.barrier()
    dist.destroy_process_group()
""")


def test_two_ranks_reach_the_full_batch_result(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT="29741")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda o: o["rank"])
    assert outs[0]["rows"] == [0, 31] and outs[1]["rows"] == [31, 61]
    for o in outs:
        assert o["proj_u"] <= 1e-9 and o["proj_q"] <= 1e-9          # the full-batch subspaces
        assert o["dw_err"] <= 1e-10                                   # the full-batch gradient
        assert o["bytes"] == (12 * 12 + 5 * 7) * 8                    # one Gram matrix and one dY^T Z, nothing else
    assert outs[0]["u_sum"] == outs[1]["u_sum"] and outs[0]["q_sum"] == outs[1]["q_sum"]


def test_shard_rows_covers_every_row_once():
    from paper_2602_23111_b200.sharded import shard_rows
    for n in (0, 1, 7, 64, 65, 1000):
        for world in (1, 2, 3, 8):
            edges = [shard_rows(n, world, r) for r in range(world)]
            assert edges[0][0] == 0 and edges[-1][1] == n
            assert all(edges[i][1] == edges[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in edges]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_rows(10, 2, 2)


def test_bench_sharded_mode_accounts_for_one_gram_and_one_middle_factor_per_group():
    """`bench.py --sharded` reports the bytes a rank sends through collectives per step; the figure it
    expects is one fp32 Gram matrix per distinct input and one fp32 dY^T Z per linear, and nothing
    when the group has one rank."""
    import sys
    sys.path.insert(0, ROOT)
    import bench
    from paper_2602_23111_b200 import inputs
    w = inputs.WORKLOADS["llama1b"]
    kr = 256
    assert bench.sharded_bytes_per_step(w, kr, 1) == 0
    d, f = w.d, w.ffn
    gram = 4 * (3 * d * d + f * f)                                  # attn-in, attn-out, mlp-in; ffn activation
    mid = 4 * 2 * kr * (4 * d + 2 * f + d)                          # q, k, v, o; up, gate; down
    assert bench.sharded_bytes_per_step(w, kr, 2) == gram + mid == bench.sharded_bytes_per_step(w, kr, 8)
    # against all-reducing dW itself (what plain data parallelism sends): the middle factors are d / (k + r) smaller
    dw = 4 * (4 * d * d + 2 * f * d + d * f)
    assert mid * (d // (2 * kr)) <= dw
