"""Host-side logic of the multi-process benchmark, run as two gloo ranks on the CPU: every rank decodes its own
sentences (replicas, no collective on the data path), the job's time is the slowest rank's and its token count
the sum; the reference arm runs on rank 0 only."""
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    src, lens = bench.sentence_inputs(rank)
    t, n = bench.reduce_max_sum(dist, torch.device("cpu"), 10.0 + 5.0 * rank, 100 + rank)
    out[rank] = (float(t), int(n), int(src.sum()), src.shape, int(lens.sum()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_sentences_and_aggregate():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29533, out), nprocs=2, join=True)
    assert out[0][:2] == (15.0, 201) and out[1][:2] == (15.0, 201)      # max over ranks, sum over ranks
    assert out[0][3] == out[1][3] == (64, 40)
    assert out[0][2] != out[1][2]                                       # different sentences per rank
    sys.path.insert(0, ROOT)
    import bench
    a, _ = bench.sentence_inputs(0)
    assert int(a.sum()) == out[0][2]                                    # and seeded


def test_single_process_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max_sum(None, None, 3.5, 7) == (3.5, 7)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_algorithmic_bytes_of_a_verification_step():
    """The byte counts behind the bench line's roofline: per-step weight bytes Ld(6d^2 + 2dF)s + Vds for the three model
    sizes (cross-attention K/V projections excluded: they run once per sentence), and the key/value terms of a step."""
    sys.path.insert(0, ROOT)
    import bench
    from paper_2205_10350_b200 import synth
    assert bench.weight_bytes(synth.BASE) == 38_404_096 * 2 == 76_808_192
    assert bench.weight_bytes(synth.BIG) == 120_848_384 * 2
    assert bench.weight_bytes(synth.TINY) == 586_752 * 4
    # one base-model step: 32 source tokens, a 16-token block on a 16-token prefix: 12 288 bytes per key/value token
    per_tok = 2 * 6 * 512 * 2
    assert per_tok == 12_288
    assert bench.step_bytes(synth.BASE, 32, 32, 16) == 76_808_192 + per_tok * (32 + 32 + 16)
    assert bench.step_bytes(synth.BASE, 0, 0, 0, n_steps=3) == 3 * 76_808_192


def test_stored_profiler_counters_expire_with_the_kernel_sources(monkeypatch):
    """The DRAM counters the bench line repeats were taken on one state of the kernel sources: they are reported while
    the sources hash to the stored digest and become null otherwise."""
    sys.path.insert(0, ROOT)
    import bench
    digest = bench.kernel_sources_digest()
    assert len(digest) == 64 and digest == bench.kernel_sources_digest()
    monkeypatch.setitem(bench.NCU_COUNTERS, "sources_sha256", digest)
    assert bench.ncu_counter("step_block40_bytes") == bench.NCU_COUNTERS["step_block40_bytes"] > bench.weight_bytes(
        __import__("paper_2205_10350_b200.synth", fromlist=["BASE"]).BASE)
    monkeypatch.setitem(bench.NCU_COUNTERS, "sources_sha256", "0" * 64)
    assert bench.ncu_counter("step_block40_bytes") is None and bench.ncu_counter("projection_bytes") is None
