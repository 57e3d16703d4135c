"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and validates shapes.  No kernel is launched here."""
import ctypes
import os
import re

import pytest

import paper_2609_32114_b200 as ha
from paper_2609_32114_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return ha.load_library()


def test_exports_match_header(lib):
    hdr = open(os.path.join(ROOT, "include", "ha_la.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(ha_la_[a-z_]+)\s*\(", hdr))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None
    assert ha.ha_la_version() >= 1
    assert ha.status_string(0) == "ok" and "workspace" in ha.status_string(3)


def test_struct_layout_matches_c(lib):
    # 10 x 4-byte scalars, 7 pointers, 2 ints, 3 pointers, size_t, pointer on LP64
    assert ctypes.sizeof(binding.ha_la_prefill_args) == 40 + 7 * 8 + 8 + 3 * 8 + 8 + 8
    assert binding.ha_la_prefill_args.q.offset == 40
    assert binding.ha_la_prefill_args.num_seqs.offset == 96
    assert binding.ha_la_prefill_args.o.offset == 104
    assert binding.ha_la_prefill_args.workspace_bytes.offset == 128


def _args(**kw):
    base = dict(variant="gdn", dtype="bf16", batch=1, seqlen=4096, hk=16, hv=16, dk=128, dv=128)
    base.update(kw)
    return ha.make_args(**base)


def test_workspace_query_and_validation(lib):
    n = ha.ha_la_prefill_workspace_bytes(_args())
    assert n > 0 and n % 256 == 0
    n5 = ha.ha_la_prefill_workspace_bytes(_args(seqlen=100000, num_seqs=8))
    assert n5 >= n
    assert ha.ha_la_prefill_path(_args(dtype="fp32", dk=64, dv=64, hk=1, hv=1, seqlen=256)) == "simt"
    assert ha.ha_la_prefill_num_launches(_args()) >= 2

    def status_of(**kw):
        out = ctypes.c_size_t(0)
        return lib.ha_la_prefill_workspace_bytes(ctypes.byref(_args(**kw)), ctypes.byref(out))

    assert status_of(variant=7) == binding.HA_LA_ERR_INVALID_ARG
    assert status_of(dtype=5) == binding.HA_LA_ERR_INVALID_ARG
    assert status_of(hv=24) == binding.HA_LA_ERR_INVALID_ARG          # not a multiple of hk
    assert status_of(batch=0) == binding.HA_LA_ERR_INVALID_ARG
    assert status_of(seqlen=-1) == binding.HA_LA_ERR_INVALID_ARG
    assert status_of(batch=2, num_seqs=3) == binding.HA_LA_ERR_INVALID_ARG
    assert status_of(dk=96) == binding.HA_LA_ERR_UNSUPPORTED
    assert status_of(chunk=32) == binding.HA_LA_ERR_UNSUPPORTED
    assert status_of(scale=float("nan")) == binding.HA_LA_ERR_INVALID_ARG
    assert lib.ha_la_prefill_workspace_bytes(None, None) == binding.HA_LA_ERR_INVALID_ARG


def test_prefill_rejects_bad_pointers_without_launching(lib):
    # every check below fails before any CUDA call is made, so this runs without a GPU
    a = _args()
    assert binding.ha_la_prefill_raw(a) == binding.HA_LA_ERR_INVALID_ARG       # null q/k/v/...
    a = _args(q=4096, k=4096, v=4096, g=4096, beta=4096, o=8192)
    assert binding.ha_la_prefill_raw(a) == binding.HA_LA_ERR_WORKSPACE         # no workspace
    a = _args(q=4096, k=4096, v=4096, g=4096, beta=4096, o=8192, workspace=4096 + 16, workspace_bytes=1 << 40)
    assert binding.ha_la_prefill_raw(a) == binding.HA_LA_ERR_WORKSPACE         # misaligned
    a = _args(q=4096, k=4096, v=4096, g=4096, beta=4096, o=8192, workspace=4096, workspace_bytes=16)
    assert binding.ha_la_prefill_raw(a) == binding.HA_LA_ERR_WORKSPACE         # too small
    a = _args(q=4098, k=4096, v=4096, g=4096, beta=4096, o=8192, workspace=4096, workspace_bytes=1 << 40)
    assert binding.ha_la_prefill_raw(a) == binding.HA_LA_ERR_INVALID_ARG       # q not 16-byte aligned
    a = _args(q=4096, k=4096, v=4096, g=4096, beta=4096, o=8192, num_seqs=2, workspace=4096, workspace_bytes=1 << 40)
    assert binding.ha_la_prefill_raw(a) == binding.HA_LA_ERR_INVALID_ARG       # packed mode without cu_seqlens


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(FileNotFoundError):
        ha.load_library(str(tmp_path / "libha_la.so"))


def test_launch_plan_for_the_benchmark_shapes(lib, monkeypatch):
    """Host-side launch planning (slice width of the sequential kernel, kernels side by side or back to back)
    for the five benchmark shapes on a 148-SM GPU (the count assumed when no GPU is present)."""
    for var in ("HA_LA_TC_NV", "HA_LA_TC_OVERLAP", "HA_LA_FORCE_SIMT"):
        monkeypatch.delenv(var, raising=False)
    plan = ha.ha_la_prefill_launch_plan
    # one 4096-token sequence, 16 heads: 64 narrow-slice CTAs beside the chunk-local kernel
    assert plan(_args()) == (32, True)
    # 16384 tokens, 32 V-heads: 128 narrow CTAs would leave no SMs; 64 CTAs of 64 channels run beside it
    assert plan(_args(seqlen=16384, hv=32)) == (64, True)
    # KDA, 8192 tokens, 32 heads: its chunk-local kernel is too slow on half of the SMs: back to back
    assert plan(_args(variant="kda", seqlen=8192, hk=32, hv=32)) == (32, False)
    # packed batch of 8 sequences (139,389 tokens, longest 30,933): more CTAs than SMs, 64-channel slices
    assert plan(_args(seqlen=139389, num_seqs=8, max_seqlen=30933)) == (64, False)
    # fp32 inputs take the CUDA-core kernel: nothing to plan
    assert plan(_args(dtype="fp32", dk=64, dv=64, hk=1, hv=1, seqlen=256)) == (0, False)
    # a single chunk cannot overlap anything; tiny problems stay back to back
    assert plan(_args(seqlen=64))[1] is False
    assert plan(_args(seqlen=512)) == (32, False)
    # the switches override the planner
    monkeypatch.setenv("HA_LA_TC_OVERLAP", "0")
    assert plan(_args()) == (32, False)
    monkeypatch.setenv("HA_LA_TC_OVERLAP", "2")
    assert plan(_args(seqlen=512)) == (32, True)
    monkeypatch.setenv("HA_LA_TC_NV", "128")
    assert plan(_args())[0] == 128
    with pytest.raises(ha.HaLaError):
        plan(_args(dk=96))
    assert lib.ha_la_prefill_launch_plan(ctypes.byref(_args()), None, None) == binding.HA_LA_ERR_INVALID_ARG


def test_workspace_follows_the_segment_plan(lib, monkeypatch):
    """The segment scratch is part of the workspace only when the plan cuts the sequences: b, the transition
    matrix (fp32) and the start state (bf16) per (sequence, V-head, segment), plus one bf16 row of 128 channels
    per (token, V-head), rounded up to 1 KiB."""
    for var in ("HA_LA_TC_NV", "HA_LA_TC_OVERLAP", "HA_LA_FORCE_SIMT", "HA_LA_TC_SEGMENTS"):
        monkeypatch.delenv(var, raising=False)
    wb, nseg = ha.ha_la_prefill_workspace_bytes, ha.ha_la_prefill_num_segments
    a = _args()                                            # the headline shape: one segment
    assert nseg(a) == 1
    plain = wb(a)
    monkeypatch.setenv("HA_LA_TC_SEGMENTS", "4")
    assert nseg(a) == 4
    rows = -(-4096 * 16 * 128 * 2 // 1024) * 1024
    assert wb(a) - plain == 16 * 4 * 128 * 128 * 10 + rows
    monkeypatch.setenv("HA_LA_TC_SEGMENTS", "1")
    assert wb(a) == plain
    monkeypatch.delenv("HA_LA_TC_SEGMENTS")
    long2 = _args(seqlen=16384, hk=2, hv=2)                # few heads, long row: the planner cuts it itself
    n = nseg(long2)
    assert n > 1
    monkeypatch.setenv("HA_LA_TC_SEGMENTS", "1")
    one = wb(long2)
    monkeypatch.delenv("HA_LA_TC_SEGMENTS")
    assert wb(long2) - one == 2 * n * 128 * 128 * 10 + 16384 * 2 * 128 * 2
