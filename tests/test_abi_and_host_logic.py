"""CPU tests: the C ABI library loads and exports what include/attn.h declares, argument
validation (which runs before any CUDA call), the FLOP counter, the rank plumbing."""
import ctypes
import os
import re
import subprocess
import sys

import numpy as np
import pytest
import torch

import paper_2605_05023_b200 as pk
from paper_2605_05023_b200 import binding
from workload_flops import row_visibility, unmasked_flops, visible_pairs
from synth_inputs import Workload, benchmark_workloads

from helpers import visible_matrix

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions(header="attn.h", prefix="attn_"):
    text = open(os.path.join(ROOT, "include", header)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(" + prefix + r"[a-z_]*)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert {"attn_fwd", "attn_fwd_host", "attn_host_workspace_bytes", "attn_status_string",
            "attn_version", "attn_launch_count", "attn_clear_cache", "attn_cache_hits",
            "attn_selftest_timeout"} <= set(names)
    lib = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert pk.version() >= 100
    assert pk.status_string(0) == "ok" and "unknown" in pk.status_string(99)


def test_descriptor_struct_matches_header_size():
    # uint32 x5, int32 x2, float x2, ptr, float x2, ptr, int32 x4, int64 x12, ptr  (natural alignment)
    assert ctypes.sizeof(binding.AttnVariantDesc) == 36 + 4 + 8 + 8 + 8 + 16 + 96 + 8


def good_desc(**kw):
    d = binding.AttnVariantDesc()
    d.struct_size = ctypes.sizeof(binding.AttnVariantDesc)
    d.dtype = binding.ATTN_BF16
    d.o_dtype = binding.ATTN_BF16
    for k, v in kw.items():
        setattr(d, k, v)
    return d


FAKE = 0x10000   # aligned, never dereferenced: every case below is rejected before any CUDA call


@pytest.mark.parametrize("args,desc,status", [
    (dict(q=0), good_desc(), 1),
    (dict(), None, 1),
    (dict(), good_desc(struct_size=8), 5),
    (dict(B=0), good_desc(), 2),
    (dict(Hq=6, Hkv=4), good_desc(), 2),
    (dict(D=96), good_desc(), 3),
    (dict(D=258), good_desc(dtype=binding.ATTN_FP32, o_dtype=binding.ATTN_FP32), 3),
    (dict(D=64), good_desc(dtype=binding.ATTN_FP32, o_dtype=binding.ATTN_BF16), 3),
    (dict(q=FAKE + 8), good_desc(), 4),
    (dict(), good_desc(normalizer=7), 5),
    (dict(), good_desc(mask_flags=64), 5),
    (dict(), good_desc(mask_flags=binding.ATTN_MASK_GLOBAL, global_len=-1), 5),
    (dict(), good_desc(mask_flags=binding.ATTN_MASK_PREFIX, prefix_len=4), 5),          # needs the causal clause
    (dict(), good_desc(mask_flags=binding.ATTN_MASK_CAUSAL | binding.ATTN_MASK_PREFIX, prefix_len=-1), 5),
    (dict(), good_desc(mask_flags=binding.ATTN_MASK_TEST_QUERY, test_query_start=4), 5),  # needs the document clause
    (dict(), good_desc(mask_flags=binding.ATTN_MASK_DOCUMENT), 5),
    (dict(B=2), good_desc(mask_flags=binding.ATTN_MASK_DOCUMENT, cu_seqlens=FAKE, num_docs=1), 2),
    (dict(Sq=64), good_desc(mask_flags=binding.ATTN_MASK_DOCUMENT, cu_seqlens=FAKE, num_docs=1), 2),
    (dict(), good_desc(scale=-1.0), 5),
    (dict(), good_desc(softcap=float("nan")), 5),
    (dict(), good_desc(q_strides=(ctypes.c_int64 * 3)(1, 1, 1)), 4),
    (dict(), good_desc(bias_slopes=FAKE + 2), 4),
])
def test_invalid_arguments_return_codes_without_launching(args, desc, status):
    a = dict(q=FAKE, k=FAKE, v=FAKE, o=FAKE, lse=FAKE, B=1, Hq=4, Hkv=4, Sq=128, Sk=128, D=128)
    a.update(args)
    before = pk.launch_count()
    rc = pk.raw_attn_fwd(a["q"], a["k"], a["v"], a["o"], a["lse"], a["B"], a["Hq"], a["Hkv"], a["Sq"], a["Sk"],
                         a["D"], desc, None)
    assert rc == status
    assert pk.launch_count() == before


def test_host_entry_point_validation():
    d = good_desc()
    assert pk.host_workspace_bytes(1, 2, 2, 128, 128, 128, d) == 4 * 65536 + 1024
    lib = binding._lib
    rc = lib.attn_fwd_host(FAKE, FAKE, FAKE, FAKE, None, 1, 2, 2, 128, 128, 128, ctypes.byref(d), FAKE, 16, None)
    assert rc == 2       # workspace too small
    rc = lib.attn_fwd_host(FAKE, FAKE, FAKE, FAKE, None, 1, 2, 2, 128, 128, 128, ctypes.byref(d), None, 1 << 30, None)
    assert rc == 1
    d2 = good_desc(q_strides=(ctypes.c_int64 * 3)(8, 8, 8))
    rc = lib.attn_fwd_host(FAKE, FAKE, FAKE, FAKE, None, 1, 2, 2, 128, 128, 128, ctypes.byref(d2), FAKE, 1 << 30, None)
    assert rc == 5


def test_host_entry_point_checks_every_argument_before_the_first_copy():
    """An argument error of the staged entry points must leave nothing on the stream: with a workspace that is
    large enough, the answer is the argument's own status (a copy would have been a CUDA call: status 6 here)."""
    lib = binding._lib
    for kw, sizes, status in [
        (dict(), dict(D=96), 3),                                   # unsupported head dimension
        (dict(normalizer=7), dict(), 5),
        (dict(dtype=9), dict(), 5),
        (dict(mask_flags=binding.ATTN_MASK_DOCUMENT), dict(), 5),  # document mask without offsets
        (dict(), dict(Hq=3, Hkv=2), 2),
    ]:
        d = good_desc(**kw)
        a = dict(B=1, Hq=2, Hkv=2, Sq=128, Sk=128, D=128)
        a.update(sizes)
        before = pk.launch_count()
        rc = lib.attn_fwd_host(FAKE, FAKE, FAKE, FAKE, None, a["B"], a["Hq"], a["Hkv"], a["Sq"], a["Sk"], a["D"],
                               ctypes.byref(d), FAKE * 16, 1 << 30, None)
        assert rc == status, (kw, sizes, rc)
        assert pk.launch_count() == before
    # the GEMM twin: N not a multiple of 8 is an alignment error, found before the copies
    rc = lib.gemm_rowsum_host(FAKE, FAKE, FAKE, FAKE, 128, 100, 64, None, FAKE * 16, 1 << 30, None)
    assert rc == 4


def test_cache_and_selftest_entry_points_validate_on_the_host():
    assert pk.clear_cache() == 0                                   # host memory only: works without a GPU
    assert pk.cache_hits() >= 0
    lib = binding._lib
    assert lib.attn_selftest_timeout(None, 1000, None, None) == 1
    assert lib.attn_selftest_timeout(FAKE + 2, 1000, None, None) == 4
    assert lib.attn_selftest_timeout(FAKE, 0, None, None) == 5
    assert lib.attn_selftest_timeout(FAKE, 10**9, None, None) == 5  # beyond 0.1 s


def test_concurrent_host_threads_get_the_same_answers():
    """Argument checks and the tensor-map cache bookkeeping from eight host threads at once."""
    import threading
    out = []

    def work():
        d = good_desc()
        codes = [pk.raw_attn_fwd(FAKE, FAKE, FAKE, FAKE, FAKE, 1, 6, 4, 128, 128, 128, d, None) for _ in range(200)]
        codes += [pk.clear_cache() for _ in range(50)]
        out.append(set(codes))

    threads = [threading.Thread(target=work) for _ in range(8)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert out == [{2, 0}] * 8


def test_cpu_tensors_are_refused():
    q = torch.zeros(1, 1, 8, 64, dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        pk.attn_fwd(q, q, q)


# ---------------------------------------------------------------------------- FLOP counter
@pytest.mark.parametrize("kw", [dict(), dict(causal=True), dict(causal=True, Sq=20, Sk=33), dict(causal=True, Sq=33, Sk=20),
                                dict(causal=True, window_left=5, window_right=0), dict(window_left=3, window_right=4),
                                dict(causal=True, cu_seqlens=(0, 1, 9, 17, 40)), dict(cu_seqlens=(0, 13, 40)),
                                dict(causal=True, window_left=6, window_right=0, cu_seqlens=(0, 13, 40)),
                                dict(causal=True, prefix_len=11), dict(causal=True, prefix_len=25, Sq=20, Sk=33),
                                dict(causal=True, cu_seqlens=(0, 1, 9, 17, 40), test_query_start=21),
                                dict(causal=True, window_left=9, window_right=0, cu_seqlens=(0, 13, 40), test_query_start=30),
                                dict(window_left=3, window_right=3, global_len=5), dict(window_left=3, window_right=3, global_len=40),
                                dict(causal=True, window_left=4, window_right=0, global_len=6, Sq=20, Sk=33),
                                dict(causal=True, cu_seqlens=(0, 9, 17, 18, 40), global_len=9)])
def test_visible_pairs_against_per_element_rule(kw):
    base = dict(name="t", B=1, Hq=1, Hkv=1, Sq=40, Sk=40, D=8)
    base.update(kw)
    w = Workload(**base)
    vis = visible_matrix(w)
    mask = dict(causal=w.causal, window_left=w.window_left, window_right=w.window_right, cu_seqlens=w.cu_seqlens,
                prefix_len=w.prefix_len, test_query_start=w.test_query_start, global_len=w.global_len)
    n = visible_pairs(w.Sq, w.Sk, **mask)
    assert n == int(vis.sum())
    pre, lo, hi = row_visibility(w.Sq, w.Sk, **mask)
    for i in range(w.Sq):
        cols = set(np.nonzero(vis[i])[0].tolist())
        assert cols == set(range(0, pre[i])) | set(range(lo[i], hi[i] + 1))
        assert pre[i] == 0 or pre[i] < lo[i]


def test_benchmark_flop_counts_closed_forms():
    w = benchmark_workloads()
    assert unmasked_flops(w["c1_fp32_causal"]) == 4 * 64 * 2 * (256 * 257 // 2)
    assert unmasked_flops(w["c2_noncausal"]) == 4 * 128 * 64 * 4096 * 4096
    assert unmasked_flops(w["c2_causal"]) == 4 * 128 * 64 * (4096 * 4097 // 2)
    # causal window of 1024 keys: rows 0..1022 see i+1 keys, the rest 1024
    assert unmasked_flops(w["c3_gqa_window_alibi"]) == 4 * 128 * 64 * (1023 * 1024 // 2 + (8192 - 1023) * 1024)
    cu = np.array(w["c5_packed_doc_causal"].cu_seqlens)
    L = np.diff(cu)
    assert unmasked_flops(w["c5_packed_doc_causal"]) == 4 * 128 * 16 * int((L * (L + 1) // 2).sum())
    assert cu[-1] == 65536 and L[:-1].min() >= 512 and L.max() <= 4096


# ---------------------------------------------------------------------------- N > 1 plumbing (gloo, 2 ranks)
WORKER = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import torch, torch.distributed as dist
from paper_2605_05023_b200.ranks import max_over_ranks, rank_seed, whole_job_throughput
from synth_inputs import Workload, make_qkv
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
w = Workload("t", 1, 1, 1, 8, 8, 16, seed=rank_seed(5, rank))
q, _, _ = make_qkv(w)
sums = [torch.zeros(1) for _ in range(world)]
dist.all_gather(sums, q.float().sum().view(1))
assert len({float(s) for s in sums}) == world, "ranks must draw different batches"
ms = max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"))
assert ms == 10.0 + 5.0 * (world - 1)
assert whole_job_throughput(100.0, ms * 1e-3, world) == world * 100.0 / (ms * 1e-3)
dist.barrier()
dist.destroy_process_group()
print("ok", rank)
"""


def test_two_rank_plumbing_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29631", str(script), ROOT]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stdout + out.stderr
    assert out.stdout.count("ok") == 2


def test_reference_arm_prints_contract_line():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
           "--steps", "1", "--warmup", "0"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr
    import json
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0


# ------------------------------------------------------------------------------------------------ GEMM + row sum
def test_library_exports_every_symbol_of_the_gemm_header():
    names = declared_functions("gemm_rowsum.h", "gemm_rowsum")
    assert set(names) == {"gemm_rowsum", "gemm_rowsum_host", "gemm_rowsum_host_workspace_bytes", "gemm_rowsum_launch_count"}
    lib = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n


def test_gemm_descriptor_struct_matches_header_size():
    assert ctypes.sizeof(binding.GemmRowsumDesc) == 4 + 4 + 8 + 8 + 8 + 8   # uint32 x2, int64 x3, ptr


def gemm_desc(**kw):
    d = binding.GemmRowsumDesc()
    d.struct_size = ctypes.sizeof(binding.GemmRowsumDesc)
    for k, v in kw.items():
        setattr(d, k, v)
    return d


@pytest.mark.parametrize("args,desc,status", [
    (dict(a=0), None, 1),
    (dict(b=0), None, 1),
    (dict(r=0), None, 1),
    (dict(M=0), None, 2),
    (dict(K=-1), None, 2),
    (dict(), gemm_desc(struct_size=8), 5),
    (dict(), gemm_desc(reserved=1), 5),
    (dict(), gemm_desc(lda=56), 2),             # leading dimension below the row length
    (dict(), gemm_desc(ldb=72), 2),
    (dict(N=100), None, 4),                     # N not a multiple of 8
    (dict(), gemm_desc(lda=68), 4),             # row stride not a multiple of 16 bytes
    (dict(a=FAKE + 2), None, 4),
    (dict(c=FAKE + 8), None, 4),
])
def test_gemm_rowsum_rejects_bad_arguments_before_any_cuda_call(args, desc, status):
    v = dict(a=FAKE, b=FAKE, c=FAKE, r=FAKE, M=128, N=128, K=64)
    v.update(args)
    rc = binding.raw_gemm_rowsum(v["a"], v["b"], v["c"], v["r"], v["M"], v["N"], v["K"], desc, None)
    assert rc == status


def test_gemm_host_workspace_size():
    n = binding.gemm_rowsum_host_workspace_bytes(100, 72, 40)
    assert n >= 100 * 40 * 2 + 40 * 72 * 2 + 100 * 72 * 2 + 100 * 4 and n % 256 == 0
    assert binding.gemm_rowsum_host_workspace_bytes(0, 8, 8) == 0
