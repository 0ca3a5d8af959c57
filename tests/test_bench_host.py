"""Host-side logic of bench.py: algorithmic work per layer, the peak table, and the multi-rank reduction (units summed
over ranks, time = the slowest rank's) exercised with two gloo ranks on CPU.  No GPU, no kernels."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from conftest import ROOT

sys.path.insert(0, ROOT)
import bench


def test_layer_work_matches_the_workload_table():
    # sweep layer: conv3x3 C = K = 64 at 56x56, batch 128: 29.6 GFLOP, 205.7 MB
    row = dict(op="conv", C=64, K=64, H=56, W=56, FH=3, FW=3, OH=56, OW=56)
    fl, by = bench.layer_work(row, 128)
    assert round(fl / 1e9, 1) == 29.6 and round(by / 1e6, 1) == 205.7
    row = dict(op="conv", C=512, K=512, H=7, W=7, FH=1, FW=1, OH=7, OW=7)
    fl, by = bench.layer_work(row, 128)
    assert round(fl / 1e9, 2) == 3.29 and round(by / 1e6, 1) == 26.7
    row = dict(op="dwconv", C=64, K=64, H=56, W=56, FH=3, FW=3, OH=56, OW=56)
    fl, by = bench.layer_work(row, 128)
    assert round(fl / 1e9, 2) == 0.46 and round(by / 1e6, 1) == 205.5
    row = dict(op="pool", C=64, K=64, H=56, W=56, FH=2, FW=2, OH=28, OW=28)
    assert round(bench.layer_work(row, 128)[1] / 1e6, 1) == 128.5
    # an accumulating convolution also reads the tensor it adds to
    row = dict(op="conv", C=16, K=16, H=32, W=32, FH=3, FW=3, OH=32, OW=32)
    assert bench.layer_work(row, 256, True)[1] - bench.layer_work(row, 256, False)[1] == 4.0 * 256 * 16 * 32 * 32


def test_mode_peaks():
    peaks = dict(hbm_gbs=6539.5, bf16_burst=1648.4, bf16_sustained=1391.6, sm_max_mhz=1965.0, source="measured")
    assert abs(bench.mode_peak_tflops("tf32", peaks) - 824.2) < 1e-6
    assert abs(bench.mode_peak_tflops("3xtf32", peaks) - 824.2 / 3) < 1e-6
    assert abs(bench.mode_peak_tflops("fp32", peaks, 148) - 148 * 128 * 2 * 1.965e9 / 1e12) < 1e-6


def _rank(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r processed 256 units in (2 + r) ms: the job did 512 units in 3 ms
    value, ms = bench.whole_job_throughput(256, 2.0 + rank, world)
    out[rank] = (value, ms)
    dist.barrier()
    dist.destroy_process_group()


def test_whole_job_throughput_two_ranks_gloo():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    for r in range(2):
        value, ms = out[r]
        assert ms == pytest.approx(3.0) and value == pytest.approx(512 / 3e-3)
    assert bench.whole_job_throughput(256, 2.0, 1) == (pytest.approx(128000.0), 2.0)
