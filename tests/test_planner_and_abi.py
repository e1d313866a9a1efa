"""CPU tests of the host logic: the library loads without a GPU and exports the whole C ABI, and the
host planner follows the parameter selection of Section III-D (pinned to the chunk splits the paper
prints in Tables V and VI)."""
import ctypes
import os
import re
import subprocess
import sys

import numpy as np
import pytest

import paper_2607_22866_b200 as gm
from paper_2607_22866_b200 import build as gm_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
B200_SMEM = 232448


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "gmagnus.h")).read()
    declared = set(re.findall(r"\b(gm_[a-z_]+)\s*\(", header)) - {"gm_alloc_fn", "gm_free_fn"}
    assert declared == set(gm.EXPORTED_SYMBOLS)
    lib = ctypes.CDLL(gm_build.build())
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings_and_no_gpu_failure_is_loud():
    lib = gm.load_library()
    assert lib.gm_status_string(0) == b"GM_OK" and lib.gm_status_string(-6) == b"GM_ERR_CAPACITY"
    import torch
    if not torch.cuda.is_available():
        # no CPU path: planning must fail with GM_ERR_CUDA, not compute anything
        rp = torch.zeros(2, dtype=torch.int64)
        A = gm.DeviceCSR(1, 1, rp, torch.zeros(0, dtype=torch.int32), torch.zeros(0, dtype=torch.float32), 0)
        with pytest.raises(gm.GmError) as ei:
            gm.binding.load_library().gm_spgemm_plan  # symbol exists
            h = ctypes.c_void_p()
            a = A._struct()
            rc = lib.gm_spgemm_plan(ctypes.byref(a), ctypes.byref(a), B200_SMEM, ctypes.byref(h))
            gm.binding._check(rc, "gm_spgemm_plan")
        assert ei.value.status == -7


def _golden_splits():
    path = os.path.join(ROOT, "tests", "golden", "planner_chunk_splits.txt")
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        lhs, rhs = line.split("->")
        fmax, required = (int(x) for x in lhs.split())
        yield fmax, required, [int(x) for x in rhs.split()]


@pytest.mark.parametrize("fmax,required,levels", list(_golden_splits()))
def test_level_split_matches_paper_tables(fmax, required, levels):
    # Tables V / VI: "required: level 0, level 1, ..." for a per-level maximum of 32 (PVC) / 64 (H200)
    W = 1024
    o = gm.PlanOpts()
    o.max_fanout, o.chunk_width = fmax, W
    p = gm.planner_params(required * W, np.float32, B200_SMEM, o)
    assert p.chunks_required == required and p.levels() == levels
    assert int(np.prod(levels)) == required
    # child(level l) = (col >> shift[l]) & (F_l - 1); concatenating the children gives col >> log2(W)
    col = required * W - 1
    idx = 0
    for l, F in enumerate(levels):
        idx = idx * F + ((col >> p.shift[l]) & (F - 1))
    assert idx == col >> 10


def test_required_chunks_double_with_scale():
    # Table VI: "the required number of chunks is tied solely to matrix scale, doubling with each scale"
    prev = None
    for scale in range(15, 25):
        p = gm.planner_params(1 << scale, np.float32, B200_SMEM)
        assert p.chunks_required == max(1, (1 << scale) // p.chunk_width)
        if prev is not None and prev >= 1 and (1 << scale) > p.chunk_width:
            assert p.chunks_required == 2 * prev
        prev = p.chunks_required


def test_b200_defaults():
    p32 = gm.planner_params(1 << 20, np.float32, B200_SMEM)
    p64 = gm.planner_params(1 << 21, np.float64, B200_SMEM)
    # dense accumulator (values + bitmap) of one block per SM: 32768 floats / 16384 doubles
    assert (p32.chunk_width, p64.chunk_width) == (32768, 16384)
    assert p32.chunks_required == 32 and p64.chunks_required == 128
    # Eq. 6 with 32 subgroups, 4-byte counters, 8-byte offsets, n_groupRows = 2, half of s_LM for elements
    s = B200_SMEM
    for sv, p in ((4, p32), (8, p64)):
        n_min = s // (2 * (4 + sv))
        raw = (s - n_min * (4 + sv) - 4) // (2 * (32 * 4 + 8))
        assert p.max_fanout == min(256, 1 << (raw.bit_length() - 1))
    assert p32.levels() == [32] and p64.levels() == [128]
    # light-row capacity: table (<= 2 slots per entry) + 64-bit sort buffer must fit s_LM; the default
    # threshold is far below it (512 products with up to 32 chunks per row, 1024 with more: beyond that the
    # sort costs more than the heavy path), the capacity itself is 8192 and can be asked for, 16384 cannot
    assert (p32.tau, p32.light_slots) == (512, 1024) and (p64.tau, p64.light_slots) == (1024, 2048)
    for sv, p in ((4, p32), (8, p64)):
        dt = np.float32 if sv == 4 else np.float64
        o = gm.PlanOpts(); o.tau = 8192
        q = gm.planner_params(1 << 20, dt, s, o)
        assert q.tau == 8192 and q.light_slots * (4 + sv) + 8192 * 8 <= s and q.light_slots >= 1.5 * 8192
        assert 2 * 8192 * 8 + 3 * 8192 * (4 + sv) > s - 1024      # the next power of two would not fit
        o.tau = 8193
        with pytest.raises(gm.GmError):
            gm.planner_params(1 << 20, dt, s, o)
    # wide column space: 2^24 columns -> 512 chunks -> two levels at the default fan-out
    p = gm.planner_params(1 << 24, np.float32, B200_SMEM)
    assert p.levels() == [256, 2]
    o = gm.PlanOpts(); o.max_fanout = 32; o.acc_ctas_per_sm = 4
    p = gm.planner_params(1 << 24, np.float32, B200_SMEM, o)
    assert p.chunk_width == 8192 and p.levels() == [32, 32, 2]


def test_column_counts_that_are_not_powers_of_two():
    o = gm.PlanOpts(); o.chunk_width = 256; o.max_fanout = 4
    for c_cols, req in [(1, 1), (255, 1), (256, 1), (257, 2), (100003, 512)]:
        p = gm.planner_params(c_cols, np.float64, B200_SMEM, o)
        assert p.chunks_required == req
        assert p.n_levels == (0 if req == 1 else int(np.ceil(np.log2(req) / 2)))


def test_planner_rejects_bad_input():
    for smem in (1000, 1 << 21):
        with pytest.raises(gm.GmError) as ei:
            gm.planner_params(1 << 20, np.float32, smem)
        assert ei.value.status == -9
    for kw in ({"chunk_width": 100}, {"chunk_width": 1 << 20}, {"max_fanout": 3}, {"tau": 1 << 20}, {"acc_ctas_per_sm": 3}):
        o = gm.PlanOpts()
        for k, v in kw.items():
            setattr(o, k, v)
        with pytest.raises(gm.GmError) as ei:
            gm.planner_params(1 << 20, np.float32, B200_SMEM, o)
        assert ei.value.status == -1


def test_batches_never_split_a_row_and_respect_the_budget():
    rng = np.random.default_rng(0)
    ip = rng.integers(100, 5000, size=400)
    prefix = np.concatenate([[0], np.cumsum(ip)]).astype(np.int64)
    bounds = gm.planner_batches(prefix, 6000)
    assert bounds[0] == 0 and bounds[-1] == 400 and all(b > a for a, b in zip(bounds, bounds[1:]))
    sizes = [prefix[b] - prefix[a] for a, b in zip(bounds, bounds[1:])]
    assert max(sizes) <= 6000
    # greedy: adding the next row would overflow
    for (a, b) in zip(bounds, bounds[1:]):
        if b < 400:
            assert prefix[b + 1] - prefix[a] > 6000
    assert gm.planner_batches(prefix, int(prefix[-1])) == [0, 400]
    with pytest.raises(gm.GmError):
        gm.planner_batches(prefix, int(ip.max()) - 1)


def test_bench_reference_arm_under_torchrun_two_ranks():
    # launch contract on CPU: two ranks (gloo is not even needed: no data-path collective); rank 0
    # alone prints one JSON line, the other rank exits 0 without work
    import json
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29731", os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--steps", "1", "--warmup", "1", "--config", "0", "--cpu-budget", "0.5"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["cpu_baseline"]["kind"] == "oracle"
    assert rec["value"] > 0 and rec["e2e"]["h2d_bytes_per_step"] == 0


def _gloo_rank(rank, world, port, out):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    ms = bench.max_over_ranks(100.0 + 50.0 * rank, world, "cpu")     # rank 1 is the slow replica
    dist.barrier()
    out.put((rank, ms, bench.replicas_value(10 ** 9, world, ms)))
    dist.destroy_process_group()


def test_replica_timing_takes_the_slowest_rank_gloo_two_ranks():
    # "replicas only": the job's step time is the maximum over ranks and the aggregate counts every rank's products
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_gloo_rank, args=(r, 2, 29733, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [150.0, 150.0]
    assert abs(got[0][2] - 2 * 2.0 * 1e9 / 0.150 / 1e9) < 1e-9 and got[0][2] == got[1][2]
