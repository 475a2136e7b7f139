"""Column-sharded layer on two CPU ranks (gloo): the shard plan, each rank's host-side packing of its own columns,
and the all-reduce that sums the partial results.  The product itself needs a GPU, so here each rank evaluates its
share with the oracle from the columns ITS OWN packed shard decodes to; the sum over ranks must be the oracle's
product of the whole layer."""
import os
import subprocess
import sys
import textwrap

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    import numpy as np, torch, torch.distributed as dist
    sys.path.insert(0, os.environ["CELTY_ROOT"])
    from oracle import celty_oracle as orc
    from paper_2608_01536_b200 import build, celty, synth
    build.build()
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    M, K = 515, 1003
    W = synth.weights(31, M, K); mask = synth.mask_bernoulli(31, M, K, 0.5)
    x = synth.activations(31, K, "laplace"); tau = synth.threshold_for_density(x, 0.5)
    shard = celty.ColumnShard(W, mask, rank=rank, world=world)          # host side only: no device
    k0, k1 = shard.k0, shard.k1
    assert k0 % 8 == 0 and 0 <= k0 <= k1 <= K
    # what the shard packed, decoded from its own image, is columns k0..k1-1 of the masked matrix
    dense = np.zeros((M, k1 - k0), np.uint16)
    for j in range(k1 - k0):
        rows, vals, runs, pad = shard.local.decode_host(j)
        dense[rows[pad == 0], j] = vals[pad == 0]
    assert np.array_equal(dense, np.where(mask[:, k0:k1] != 0, W.view(np.uint16)[:, k0:k1], 0))
    # this rank's partial result, from those columns and its slice of x
    part, _ = orc.masked_gemv(dense, (dense & 0x7FFF) != 0, x[k0:k1], tau)
    bounds = torch.tensor([k0, k1], dtype=torch.int64)
    allb = [torch.zeros(2, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(allb, bounds)
    y = torch.from_numpy(part.copy())
    dist.all_reduce(y, op=dist.ReduceOp.SUM)                            # the exchange step of the sharded layer
    if rank == 0:
        assert allb[0][0] == 0 and allb[-1][1] == K
        assert all(int(a[1]) == int(b[0]) for a, b in zip(allb, allb[1:]))
        y_ref, a_ref = orc.masked_gemv(W, mask, x, tau)
        assert np.all(np.abs(y.numpy() - y_ref) <= 1e-12 * a_ref + 1e-300)
        print("SHARDS_OK", [tuple(int(v) for v in b) for b in allb])
    dist.destroy_process_group()
""")


def test_two_column_shards_sum_to_the_layer(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, CELTY_ROOT=ROOT, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29741", str(script)],
                         capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-3000:]
    assert "SHARDS_OK [(0, 504), (504, 1003)]" in out.stdout


def test_shard_plan_properties():
    sys.path.insert(0, ROOT)
    from paper_2608_01536_b200 import build, celty
    build.build()
    for K in (1, 7, 8, 9, 1003, 4096, 28672):
        for world in (1, 2, 3, 8, 64):
            ranges = [celty.shard_columns(K, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == K
            assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
            assert all(a % 8 == 0 for a, b in ranges if b > a)      # an empty shard has no slice of x to align
            sizes = [b - a for a, b in ranges]
            assert max(sizes) - min(sizes) <= 15            # whole groups of 8 columns, the last one may be short
