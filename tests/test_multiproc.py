"""N > 1 bookkeeping with two gloo ranks on CPU: independent batches per rank,
max-over-ranks timing, whole-job throughput = all ranks' work / slowest rank."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist

    from paper_2608_25683_b200 import binding, dist_util
    from paper_2608_25683_b200.workloads import make_workload

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = make_workload("c2", dist_util.rank_seed(2000, rank), scale_len=0.1)
    plan = binding.Plan(w.parent, w.seg_len, w.group_block_size, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype)
    flops = 14.0 * w.head_dim * w.n_q_heads * plan.view["tree_pairs"]
    ms = 2.0 + rank  # rank 1 is the slow one
    ms_max, flops_all = dist_util.aggregate(ms, flops)
    val = dist_util.whole_job_tflops(ms, flops)
    out.put((rank, flops, ms_max, flops_all, val, plan.view["T"]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_gloo(lib):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29000 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, f0, m0, fa0, v0, T0), (r1, f1, m1, fa1, v1, T1) = res
    assert T0 != T1, "ranks must draw independent batches"
    assert m0 == m1 == 3.0
    assert fa0 == fa1 == f0 + f1
    assert abs(v0 - (f0 + f1) / 3.0e-3 / 1e12) < 1e-9 and v0 == v1
