"""ha_la_prefill_noalloc: the entry point for callers that cannot allocate or pass scratch memory
(operator hooks that must stay out of a framework's allocator, runtimes with a frozen memory pool).

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.  The test calls the new entry point through the C ABI twice in a row, on two
different problems, and checks each result against ha_la_prefill on the same inputs within the
library's own tolerance; the second call also shows that whatever the first call left in the
library's fixed scratch array does no harm."""
import numpy as np
import pytest

from paper_2609_32114_b200 import synth
from tests import helpers

pytestmark = pytest.mark.gpu


def _both(inp):
    import torch
    import paper_2609_32114_b200 as ha

    w = inp["workload"]
    d = helpers.to_device(inp)
    common = dict(variant=w.variant, h0=d["h0"], cu_seqlens=d["cu_seqlens"], max_seqlen=d["max_seqlen"])
    # reference: the existing entry point with a caller-provided workspace
    o_ref, hT_ref, st_ref, _ = ha.ha_la_prefill(d["q"], d["k"], d["v"], d["g"], d["beta"], **common)
    # new entry point: same tensors, poisoned outputs, NO workspace (null pointer, zero bytes)
    args, keep = ha.prepare_args(d["q"], d["k"], d["v"], d["g"], d["beta"], **common)
    keep["o"].fill_(float("nan"))
    keep["hT"].fill_(float("nan"))
    args.workspace = None
    args.workspace_bytes = 0
    rc = ha.ha_la_prefill_noalloc(args, torch.cuda.current_stream().cuda_stream)
    assert rc == 0, ha.status_string(rc)
    torch.cuda.synchronize()
    assert int(st_ref.item()) == 0 and int(keep["status_word"].item()) == 0
    tol = helpers.TOL[w.dtype]
    o_a, o_b = keep["o"].float().cpu().numpy(), o_ref.float().cpu().numpy()
    h_a, h_b = keep["hT"].cpu().numpy(), hT_ref.cpu().numpy()
    assert np.isfinite(o_a).all() and np.isfinite(h_a).all()
    assert np.abs(o_a - o_b).max() <= tol * np.abs(o_b).max()
    assert np.abs(h_a - h_b).max() <= tol * np.abs(h_b).max()
    # ... and against the CPU oracle (with bf16 inputs and d = 128 ha_la_prefill runs the tensor-core kernels,
    # so this entry point is the only caller of the CUDA-core kernel for that shape)
    o_orc, h_orc = helpers.run_oracle(inp)
    assert helpers.rel_max_err(o_a.reshape(o_orc.shape), o_orc) <= tol
    assert helpers.rel_max_err(h_a.reshape(h_orc.shape), h_orc) <= tol


def test_noalloc_matches_prefill_twice_in_a_row():
    from paper_2609_32114_b200 import build
    import paper_2609_32114_b200 as ha

    build.build()
    assert 0 < ha.ha_la_prefill_noalloc_scratch_bytes() <= 256 * 1024
    # call 1: a packed batch with ragged and empty sequences (many chunk slots, several sequences)
    w1 = synth.shrink(synth.WORKLOADS["gdn_varlen"], seq_lens=[300, 0, 65, 700, 1], hk=2, hv=2)
    _both(synth.make_inputs(w1, seed=41))
    # call 2, straight after: a smaller, differently shaped problem (fp32, one sequence, d = 64)
    _both(synth.make_inputs(synth.WORKLOADS["gdn_fp32_small"], seed=42))


def test_noalloc_rejects_problems_beyond_its_scratch():
    import paper_2609_32114_b200 as ha
    from paper_2609_32114_b200 import binding

    # 2,000,000 tokens need 31,250 chunk slots > 16,384; refused before any pointer is touched beyond null checks
    a = ha.make_args(variant="gdn", dtype="bf16", batch=1, seqlen=2_000_000, hk=1, hv=1, dk=64, dv=64,
                     q=4096, k=4096, v=4096, g=4096, beta=4096, o=8192)
    assert ha.ha_la_prefill_noalloc(a) == binding.HA_LA_ERR_TOO_LARGE
    assert "scratch" in ha.status_string(binding.HA_LA_ERR_TOO_LARGE)
    a = ha.make_args(variant="gdn", dtype="bf16", batch=1, seqlen=4096, hk=1, hv=1, dk=64, dv=64, num_seqs=2000,
                     q=4096, k=4096, v=4096, g=4096, beta=4096, o=8192, cu_seqlens=4096)
    assert ha.ha_la_prefill_noalloc(a) == binding.HA_LA_ERR_TOO_LARGE


def test_noalloc_accepts_its_documented_limits():
    """Exactly 1024 sequences and 16384 chunk slots is inside the documented limits: the size check must pass
    (the call is then refused for its null pointers, before anything is launched)."""
    import paper_2609_32114_b200 as ha
    from paper_2609_32114_b200 import binding

    seqlen = 16384 * 64 - 63 * 1024                    # (seqlen + 63 * num_seqs) / 64 == 16384 chunk slots
    a = ha.make_args(variant="gdn", dtype="bf16", batch=1, seqlen=seqlen, hk=1, hv=1, dk=64, dv=64, num_seqs=1024)
    assert ha.ha_la_prefill_noalloc(a) == binding.HA_LA_ERR_INVALID_ARG      # null q, k, ...: sizes were accepted
    a = ha.make_args(variant="gdn", dtype="bf16", batch=1, seqlen=seqlen + 64, hk=1, hv=1, dk=64, dv=64,
                     num_seqs=1024, q=4096, k=4096, v=4096, g=4096, beta=4096, o=8192, cu_seqlens=4096)
    assert ha.ha_la_prefill_noalloc(a) == binding.HA_LA_ERR_TOO_LARGE
