"""GPU parity: the CUDA library (through its C ABI) against the CPU fp64 oracle, element by element,
on the same seeded inputs.  Tolerances are the stated ones (helpers.TOL): max|err|/max|ref|
<= 2e-2 for bf16 inputs, <= 1e-4 for fp32, for o and for hT separately."""
import dataclasses

import numpy as np
import pytest

from paper_2609_32114_b200 import synth
from tests import helpers

pytestmark = pytest.mark.gpu

W = synth.WORKLOADS


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2609_32114_b200 import build
    build.build()


def test_config1_gdn_fp32_exact_shape():
    inp = synth.make_inputs(W["gdn_fp32_small"])
    res = helpers.check_parity(inp)
    assert res["o_err"] < 1e-4 and res["hT_err"] < 1e-4


@pytest.mark.parametrize("T", [1, 63, 64, 65, 1000])
def test_gdn_bf16_small_ragged(T):
    w = synth.shrink(W["gdn_layer_4k"], seq_lens=[T], hk=2, hv=2)
    helpers.check_parity(synth.make_inputs(w, seed=11 + T))


@pytest.mark.parametrize("gate_shift", [-4.0, None])
def test_gdn_bf16_slow_decay(gate_shift):
    """Slow or no decay keeps old chunks visible, which is what exercises the inter-chunk state."""
    w = synth.shrink(W["gdn_layer_4k"], seq_lens=[1500], hk=2, hv=2, gate_shift=gate_shift or 0.0, h0_std=0.02)
    inp = synth.make_inputs(w, seed=5)
    if gate_shift is None:
        inp["g"][:] = 0
    helpers.check_parity(inp)


def test_gdn_fp32_d128_and_scale():
    w = dataclasses.replace(W["gdn_fp32_small"], dk=128, dv=128, seq_lens=(300,), hk=2, hv=2, h0_std=0.02)
    helpers.check_parity(synth.make_inputs(w, seed=3), scale=0.25)


def test_gva_small():
    w = synth.shrink(W["gdn_gva_16k"], seq_lens=[700], hk=2, hv=4)
    helpers.check_parity(synth.make_inputs(w, seed=7))


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_kda_small(dtype):
    w = synth.shrink(W["kda_8k"], seq_lens=[330], hk=2, hv=2, dtype=dtype, h0_std=0.02)
    helpers.check_parity(synth.make_inputs(w, seed=9))


def test_kda_slow_decay():
    w = synth.shrink(W["kda_8k"], seq_lens=[700], hk=1, hv=2, gate_shift=-4.0)
    helpers.check_parity(synth.make_inputs(w, seed=10))


def test_kda_extreme_decay_inside_a_block():
    """A few tokens forget almost everything in some channels (log-gate -90: a factor 2^-130).  Inside their
    16-token block the tensor-core factorisation of the decay would need 2^+130, so the kernel has to take
    its element-wise evaluation for those diagonal blocks; everything else stays on the tensor cores."""
    w = synth.shrink(W["kda_8k"], seq_lens=[300], hk=1, hv=2)
    inp = synth.make_inputs(w, seed=12)
    g = inp["g"]
    assert g.ndim == 3 and g.shape[-1] == 128
    for tok in (5, 37, 70, 71, 200):
        g[tok, :, ::7] = -90.0
    helpers.check_parity(inp)


@pytest.mark.parametrize("variant,dtype", [("gdn", "bf16"), ("kda", "bf16"), ("kda", "fp32")])
def test_head_dim_64_every_variant_and_dtype(variant, dtype):
    """d_k = d_v = 64 runs on the CUDA-core kernel for every variant and input type (fp32 GDN is workload 1)."""
    import paper_2609_32114_b200 as ha

    base = W["gdn_layer_4k"] if variant == "gdn" else W["kda_8k"]
    w = synth.shrink(base, seq_lens=[130, 0, 257], hk=2, hv=4, dk=64, dv=64, dtype=dtype, h0_std=0.02,
                     gate_shift=0.0, varlen=True)
    inp = synth.make_inputs(w, seed=71)
    a = ha.make_args(variant=variant, dtype=dtype, batch=1, seqlen=inp["T"], hk=2, hv=4, dk=64, dv=64, num_seqs=3)
    assert ha.ha_la_prefill_path(a) == "simt"
    helpers.check_parity(inp)


@pytest.mark.parametrize("variant", ["gdn", "kda"])
@pytest.mark.parametrize("knorm,bmax", [(0.5, 1.0), (2.0, 0.45)])
def test_tc_keys_not_normalised(variant, knorm, bmax):
    """Keys of norm 0.5 and 2 on the tensor-core path (every other case has unit keys).  beta is scaled so that
    beta |k|^2 stays below 2, the delta rule's own stability bound; slow decay keeps the state in play."""
    base = W["gdn_layer_4k"] if variant == "gdn" else W["kda_8k"]
    w = synth.shrink(base, seq_lens=[900], hk=2, hv=2, gate_shift=-3.0, h0_std=0.02)
    inp = synth.make_inputs(w, seed=73)
    inp["k"] = synth.round_to_bf16(inp["k"] * np.float32(knorm))
    inp["beta"] = (inp["beta"] * np.float32(bmax)).astype(np.float32)
    helpers.check_parity(inp)


def test_tc_solve_overflow_is_reported():
    """Keys far outside the delta rule's stable range (beta |k|^2 of several hundred) make (I + A)^-1 leave the
    fp16 range the tensor-core solve works in: the call must say so through the status word
    (HA_LA_ERR_DEVICE_CHECK), not return silently wrong numbers."""
    w = synth.shrink(W["gdn_layer_4k"], seq_lens=[256], hk=1, hv=1, gate_shift=-6.0)
    inp = synth.make_inputs(w, seed=79)
    rng = np.random.default_rng(3)
    k = 30.0 * inp["k"] + 20.0 * rng.standard_normal(inp["k"].shape[-1]).astype(np.float32) / np.sqrt(128.0)
    inp["k"] = synth.round_to_bf16(k.astype(np.float32))      # strongly correlated keys of norm ~ 36
    inp["beta"][:] = 1.0
    _, _, status = helpers.run_gpu(inp)
    assert status == 6                                               # HA_LA_ERR_DEVICE_CHECK


def test_varlen_small_with_empty_and_tiny_sequences():
    w = synth.shrink(W["gdn_varlen"], seq_lens=[70, 0, 129, 64, 5, 1, 600], hk=2, hv=2)
    inp = synth.make_inputs(w, seed=13)
    o, hT, status = helpers.run_gpu(inp)
    assert status == 0
    np.testing.assert_array_equal(hT[1], inp["h0"][1].astype(np.float64))     # empty sequence: hT = h0
    helpers.check_parity(inp)


def test_batched_equal_length_rows():
    w = synth.shrink(W["gdn_layer_4k"], seq_lens=[200, 200, 200], hk=2, hv=2, h0_std=0.02)
    helpers.check_parity(synth.make_inputs(w, seed=17))


def test_split_resume_and_in_place_state():
    """Prefill [0,T1) then [T1,T) with h0 := hT (same buffer) equals one call: only the state crosses."""
    import torch
    import paper_2609_32114_b200 as ha

    w = synth.shrink(W["gdn_layer_4k"], seq_lens=[500], hk=2, hv=2)
    inp = synth.make_inputs(w, seed=19)
    d = helpers.to_device(inp)
    o_full, hT_full, st, _ = ha.ha_la_prefill(d["q"], d["k"], d["v"], d["g"], d["beta"])
    T1 = 203
    cut = lambda t, a, b: t[:, a:b].contiguous()
    state = torch.zeros_like(hT_full)
    oa, _, st1, _ = ha.ha_la_prefill(*(cut(d[x], 0, T1) for x in ("q", "k", "v", "g", "beta")), h0=state, hT=state)
    ob, _, st2, _ = ha.ha_la_prefill(*(cut(d[x], T1, 500) for x in ("q", "k", "v", "g", "beta")), h0=state, hT=state)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and int(st1.item()) == 0 and int(st2.item()) == 0
    o_split = torch.cat([oa, ob], dim=1).float().cpu().numpy()
    o_ref = o_full.float().cpu().numpy()
    scale_o = np.abs(o_ref).max()
    assert np.abs(o_split - o_ref).max() / scale_o <= 2e-2
    h_ref = hT_full.cpu().numpy()
    assert np.abs(state.cpu().numpy() - h_ref).max() / np.abs(h_ref).max() <= 2e-2
    # ... and both equal the oracle's single run
    o_orc, h_orc = helpers.run_oracle(inp)
    assert helpers.rel_max_err(o_split[0], o_orc) <= 2e-2
    assert helpers.rel_max_err(state.cpu().numpy()[0:1].reshape(h_orc.shape), h_orc) <= 2e-2


@pytest.mark.parametrize("overlap", ["0", "2"])
@pytest.mark.parametrize("variant", ["gdn", "kda"])
def test_dependent_calls_queued_with_nothing_between_them(variant, overlap, monkeypatch):
    """A sequence prefilled piece by piece, the state handed on in place (h0 = hT = one buffer), every call
    prepared beforehand and then queued directly behind the previous one: the next call's first kernel is
    launched and set up under the previous call's tail and must still see that call's state.  The whole
    round is repeated so that the first piece follows the last piece of the round before."""
    import torch
    import paper_2609_32114_b200 as ha

    monkeypatch.setenv("HA_LA_TC_OVERLAP", overlap)
    base = W["gdn_layer_4k"] if variant == "gdn" else W["kda_8k"]
    w = synth.shrink(base, seq_lens=[2560], hk=2, hv=2, gate_shift=-3.0)      # slow decay: the state matters
    inp = synth.make_inputs(w, seed=131)
    d = helpers.to_device(inp)
    pieces = [(0, 640), (640, 1024), (1024, 1100), (1100, 2048), (2048, 2560)]
    state = torch.zeros((1, 2, 128, 128), dtype=torch.float32, device="cuda")
    o = torch.zeros_like(d["v"])
    calls = []
    for a, b in pieces:
        cut = lambda t: t[:, a:b].contiguous()
        o_piece = torch.empty_like(cut(d["v"]))
        args, keep = ha.prepare_args(cut(d["q"]), cut(d["k"]), cut(d["v"]), cut(d["g"]), cut(d["beta"]),
                                     variant=variant, h0=state, hT=state, o=o_piece)
        calls.append((args, keep, a, b))
    stream = torch.cuda.current_stream().cuda_stream
    torch.cuda.synchronize()
    for rnd in range(3):
        state.zero_()
        for args, keep, a, b in calls:                       # nothing but these launches goes on the stream
            assert ha.ha_la_prefill_raw(args, stream) == 0
    torch.cuda.synchronize()
    for args, keep, a, b in calls:
        assert int(keep["status_word"].item()) == 0
        o[:, a:b] = keep["o"]
    o_ref, h_ref = helpers.run_oracle(inp)
    assert helpers.rel_max_err(o[0].float().cpu().numpy(), o_ref) <= 2e-2
    assert helpers.rel_max_err(state.cpu().numpy().reshape(h_ref.shape), h_ref) <= 2e-2


@pytest.mark.parametrize("shape", ["side_by_side", "back_to_back", "segments", "packed"])
def test_call_captured_in_a_cuda_graph(shape):
    """A call captured by stream capture and replayed on new contents of the same buffers: every replay must equal
    an ordinary call on those contents.  (Side by side, the ready flags a replay leaves behind carry the very
    epoch the next replay runs with: under capture the call clears them first.)"""
    import torch
    import paper_2609_32114_b200 as ha

    kw = {"side_by_side": dict(seq_lens=[2048], hk=16, hv=16), "back_to_back": dict(seq_lens=[1000], hk=4, hv=4),
          "segments": dict(seq_lens=[8192], hk=2, hv=2), "packed": dict(seq_lens=[300, 0, 700, 64], hk=2, hv=4, varlen=True)}[shape]
    w = synth.shrink(W["gdn_varlen"] if shape == "packed" else W["gdn_layer_4k"], h0_std=0.02, **kw)
    dev = [helpers.to_device(synth.make_inputs(w, seed=s)) for s in (171, 172)]
    buf = {k: (v.clone() if hasattr(v, "clone") else v) for k, v in dev[0].items()}
    a, keep = ha.prepare_args(buf["q"], buf["k"], buf["v"], buf["g"], buf["beta"], variant=w.variant, h0=buf["h0"],
                              cu_seqlens=buf["cu_seqlens"], max_seqlen=buf["max_seqlen"])
    nv, conc = ha.ha_la_prefill_launch_plan(a)
    assert conc == (shape == "side_by_side") and (ha.ha_la_prefill_num_segments(a) > 1) == (shape == "segments")
    names = [k for k in ("q", "k", "v", "g", "beta", "h0") if buf[k] is not None]
    side = torch.cuda.Stream()
    ref = []
    with torch.cuda.stream(side):
        for d in dev:                                        # ordinary calls: the references (and the warm-up)
            for k in names:
                buf[k].copy_(d[k])
            assert ha.ha_la_prefill_raw(a, side.cuda_stream) == 0
            side.synchronize()
            ref.append((keep["o"].clone(), keep["hT"].clone()))
    assert not torch.equal(ref[0][0], ref[1][0])
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        assert ha.ha_la_prefill_raw(a, torch.cuda.current_stream().cuda_stream) == 0
    for rep in range(6):
        which = (rep + 1) % 2
        for k in names:
            buf[k].copy_(dev[which][k])
        keep["o"].zero_()
        keep["hT"].zero_()
        g.replay()
        torch.cuda.synchronize()
        assert int(keep["status_word"].item()) == 0
        assert torch.equal(keep["o"], ref[which][0]) and torch.equal(keep["hT"], ref[which][1]), f"replay {rep}"
    helpers.check_parity(synth.make_inputs(w, seed=171))     # ... and the ordinary call equals the oracle


@pytest.mark.parametrize("seed", [21, 22, 23])
def test_random_shapes_and_launch_modes(seed, monkeypatch):
    """A seeded sweep over what the planner can be made to do: variant, packed or batched sequences with lengths
    around the chunk boundaries (empty ones included), head counts and grouping, gate strength, initial state,
    slice width, launch mode, segment count, output scale -- each case against the oracle."""
    import random

    rng = random.Random(seed)
    for it in range(14):
        variant = rng.choice(["gdn", "kda"])
        nseq = rng.choice([1, 1, 2, 3, 5])
        lens = [rng.choice([0, 1, 63, 64, 65, 127, 128, 129, 200, 511, 700, 1000, 1537]) for _ in range(nseq)]
        if sum(lens) == 0:
            lens[0] = 77
        hk = rng.choice([1, 2, 4])
        hv = hk * rng.choice([1, 1, 2])
        packed = rng.choice([True, True, False])
        if not packed:
            lens = [max(lens[0], 1)] * nseq
        base = W["gdn_varlen"] if variant == "gdn" else W["kda_8k"]
        w = synth.shrink(base, seq_lens=lens, hk=hk, hv=hv, gate_shift=rng.choice([-4.0, -2.0, 0.0, 2.0]),
                         h0_std=rng.choice([0.0, 0.02]), varlen=packed)
        nv = rng.choice(["", "32", "64", "128"])
        ov = rng.choice(["", "0", "2"])
        sg = rng.choice(["", "", "2", "4", "8"]) if nv != "128" else ""
        for key, val in (("HA_LA_TC_NV", nv), ("HA_LA_TC_OVERLAP", ov), ("HA_LA_TC_SEGMENTS", sg)):
            if val:
                monkeypatch.setenv(key, val)
            else:
                monkeypatch.delenv(key, raising=False)
        inp = synth.make_inputs(w, seed=1000 * seed + it)
        try:
            helpers.check_parity(inp, scale=rng.choice([1.0, 0.5]))
        except AssertionError as e:
            raise AssertionError(f"case {it}: {variant} lens={lens} hk={hk} hv={hv} packed={packed} nv={nv!r} "
                                 f"overlap={ov!r} segments={sg!r}: {e}") from e


def test_run_to_run_determinism():
    w = synth.shrink(W["gdn_layer_4k"], seq_lens=[777], hk=2, hv=4)
    inp = synth.make_inputs(w, seed=23)
    o1, h1, _ = helpers.run_gpu(inp)
    o2, h2, _ = helpers.run_gpu(inp)
    np.testing.assert_array_equal(o1, o2)
    np.testing.assert_array_equal(h1, h2)


def test_bad_cu_seqlens_reports_device_check():
    import torch

    w = synth.shrink(W["gdn_varlen"], seq_lens=[100, 50], hk=1, hv=1)
    inp = synth.make_inputs(w, seed=29)
    inp["cu_seqlens"] = np.array([0, 120, 100], dtype=np.int32)     # decreasing; last entry != T
    o, hT, status = helpers.run_gpu(inp)
    assert status == 6                                               # HA_LA_ERR_DEVICE_CHECK
    torch.cuda.synchronize()


@pytest.mark.parametrize("variant", ["gdn", "kda"])
@pytest.mark.parametrize("nseg,nv", [(2, 32), (4, 32), (2, 64), (8, 64)])
def test_segment_parallel_state_passing(variant, nseg, nv, monkeypatch):
    """A sequence's chunks cut into segments that are walked at the same time (later segments from a zero state and
    from the identity, then one affine fix-up per segment).  Slow decay and no decay at all keep the start state of
    every segment in play -- a wrong start state shows there -- with an initial state, a ragged tail, segment
    boundaries that do not divide the chunk count, and batched rows."""
    import paper_2609_32114_b200 as ha

    monkeypatch.setenv("HA_LA_TC_SEGMENTS", str(nseg))
    monkeypatch.setenv("HA_LA_TC_NV", str(nv))
    base = W["gdn_layer_4k"] if variant == "gdn" else W["kda_8k"]
    for lens, shift in (([1100], -4.0), ([700, 700], None), ([130], 2.0)):
        w = synth.shrink(base, seq_lens=lens, hk=1, hv=2, gate_shift=shift or 0.0, h0_std=0.05)
        inp = synth.make_inputs(w, seed=91 + nseg)
        if shift is None:
            inp["g"][:] = 0
        a = ha.make_args(variant=variant, dtype="bf16", batch=len(lens), seqlen=lens[0], hk=1, hv=2, dk=128, dv=128)
        want = nseg if nseg <= (lens[0] + 63) // 64 else None
        if want:
            assert ha.ha_la_prefill_num_segments(a) == nseg
        helpers.check_parity(inp)


@pytest.mark.parametrize("variant", ["gdn", "kda"])
@pytest.mark.parametrize("nseg", [2, 4])
def test_segments_on_a_packed_batch(variant, nseg, monkeypatch):
    """Packed batches are never cut into segments by the planner, but the kernels take them (HA_LA_TC_SEGMENTS
    forces it): every sequence is cut into the same number of segments, so short and empty sequences end up with
    empty segments, and there are more runs than SMs."""
    monkeypatch.setenv("HA_LA_TC_SEGMENTS", str(nseg))
    base = W["gdn_varlen"] if variant == "gdn" else W["kda_8k"]
    w = synth.shrink(base, seq_lens=[700, 0, 65, 1500, 130, 1], hk=2, hv=4, gate_shift=-3.0, h0_std=0.05, varlen=True)
    inp = synth.make_inputs(w, seed=97 + nseg)
    o, hT, status = helpers.run_gpu(inp)
    assert status == 0
    np.testing.assert_array_equal(hT[1], inp["h0"][1].astype(np.float64))     # empty sequence: hT = h0 exactly
    helpers.check_parity(inp)


def test_segments_chosen_only_where_every_run_gets_an_sm():
    """Host side of the planner: the headline layer (16 heads) keeps one segment, a long sequence with two heads
    is cut up, packed batches never are."""
    import paper_2609_32114_b200 as ha

    mk = lambda **kw: ha.make_args(**dict(dict(variant="gdn", dtype="bf16", batch=1, seqlen=4096, hk=16, hv=16,
                                               dk=128, dv=128), **kw))
    assert ha.ha_la_prefill_num_segments(mk()) == 1
    assert ha.ha_la_prefill_num_segments(mk(seqlen=16384, hk=2, hv=2)) > 1
    assert ha.ha_la_prefill_num_segments(mk(seqlen=16384, hk=2, hv=2, num_seqs=2)) == 1


def test_bounded_wait_runs_out_and_reports_timeout():
    """Every device-side wait is bounded.  The test hook launches the sequential kernel alone, waiting per chunk for
    flags that nothing publishes, with a limit of a few thousand polls: the wait must run out, the status word must
    say HA_LA_ERR_TIMEOUT, the kernel must exit normally, and the library must work as before afterwards."""
    import torch
    import paper_2609_32114_b200 as ha
    from paper_2609_32114_b200 import binding

    w = synth.shrink(W["gdn_layer_4k"], seq_lens=[300], hk=1, hv=2)
    inp = synth.make_inputs(w, seed=83)
    d = helpers.to_device(inp)
    args, keep = ha.prepare_args(d["q"], d["k"], d["v"], d["g"], d["beta"], variant="gdn")
    keep["workspace"].zero_()
    rc = ha.ha_la_debug_wait_timeout(args, torch.cuda.current_stream().cuda_stream, 3000)
    assert rc == 0, ha.status_string(rc)
    torch.cuda.synchronize()                                   # returns: nothing hangs, nothing faults
    assert int(keep["status_word"].item()) == binding.HA_LA_ERR_TIMEOUT
    helpers.check_parity(inp)                                  # the next ordinary call is unaffected


# ---------------------------------------------------------------- full-size configurations, every head

@pytest.mark.parametrize("name", ["gdn_layer_4k", "gdn_gva_16k", "kda_8k", "gdn_varlen"])
def test_full_size_all_heads(name):
    """Full-size workload in the launch configuration the bench times, compared with the oracle on every
    (sequence, V-head) pair and every token (the oracle needs a few seconds per workload)."""
    inp = synth.make_inputs(W[name])
    res = helpers.check_parity(inp)
    print(name, res)


@pytest.mark.parametrize("variant,nv,hv", [("gdn", 32, 16), ("gdn", 64, 16), ("kda", 64, 32), ("kda", 32, 16)])
def test_consumed_images_dropped_from_l2(variant, nv, hv, monkeypatch):
    """Side by side with operand images larger than L2, the chain kernel drops the images it has consumed
    from L2 (a slice its own rows, the last slice of a head the shared ones, counted in the chunk's flag): every
    head against the oracle, with four slices (32 channels) and two (64) per head, both variants; twice in a row
    on one workspace, so that the second call finds the first call's counts in the flags."""
    import torch
    import paper_2609_32114_b200 as ha

    monkeypatch.setenv("HA_LA_TC_NV", str(nv))
    monkeypatch.setenv("HA_LA_TC_OVERLAP", "2")
    monkeypatch.setenv("HA_LA_TC_SEGMENTS", "1")
    base = W["gdn_layer_4k"] if variant == "gdn" else W["kda_8k"]
    w = synth.shrink(base, seq_lens=[8192], hk=hv, hv=hv, h0_std=0.02)      # 128 chunks x hv heads x 64.8 KiB
    inp = synth.make_inputs(w, seed=151 + nv)
    d = helpers.to_device(inp)
    a, keep = ha.prepare_args(d["q"], d["k"], d["v"], d["g"], d["beta"], variant=variant, h0=d["h0"])
    assert ha.ha_la_prefill_launch_plan(a) == (nv, True)
    stream = torch.cuda.current_stream().cuda_stream
    o_ref, h_ref = helpers.run_oracle(inp)
    for rep in range(2):
        keep["o"].zero_()
        keep["hT"].zero_()
        assert ha.ha_la_prefill_raw(a, stream) == 0
        torch.cuda.synchronize()
        assert int(keep["status_word"].item()) == 0
        assert helpers.rel_max_err(keep["o"][0].float().cpu().numpy(), o_ref) <= 2e-2
        assert helpers.rel_max_err(keep["hT"].cpu().numpy().reshape(h_ref.shape), h_ref) <= 2e-2


def test_tensors_beyond_two_gib():
    """One 270,000-token sequence with 32 V-heads on one q/k head: v and o are 2.2 GB each, so element offsets pass
    2^30 and byte offsets 2^31 (index arithmetic in 32 bits would wrap), the workspace is 8.8 GB, and a ragged last
    chunk sits at the far end.  Every head against the oracle (about a minute, half of it drawing the inputs).
    Run once by hand at 530,000 tokens (4.3 GB per tensor, past 2^31 elements) and for KDA with a 4.4 GB gate
    tensor: both within the same tolerance."""
    w = synth.shrink(W["gdn_gva_16k"], seq_lens=[270000], hk=1, hv=32, h0_std=0.02)
    inp = synth.make_inputs(w, seed=5)
    assert inp["v"].size * 2 > 2 ** 31
    helpers.check_parity(inp)


@pytest.mark.parametrize("variant", ["gdn", "kda"])
@pytest.mark.parametrize("nv", [32, 64, 128])
def test_tc_every_slice_width(nv, variant, monkeypatch):
    """The tensor-core chain kernel at each value-slice width (normally chosen from the launch size): full
    chunks (stored as tiles by the wider slices) and ragged last chunks (stored row by row) in one batch."""
    import paper_2609_32114_b200 as ha

    monkeypatch.setenv("HA_LA_TC_NV", str(nv))
    base = W["gdn_varlen"] if variant == "gdn" else W["kda_8k"]
    w = synth.shrink(base, seq_lens=[130, 700, 64], hk=2, hv=4, gate_shift=-1.0, varlen=True)
    inp = synth.make_inputs(w, seed=31 + nv)
    a = ha.make_args(variant=variant, dtype="bf16", batch=1, seqlen=inp["T"], hk=2, hv=4, dk=128, dv=128, num_seqs=3)
    assert ha.ha_la_prefill_path(a) == "tc"
    helpers.check_parity(inp)


@pytest.mark.parametrize("case", ["gdn", "kda", "varlen", "gdn_nv64", "kda_nv64", "gdn_nv128", "kda_nv128"])
def test_concurrent_prep_and_chain_mode(case, monkeypatch):
    """Concurrent mode (chosen by the launch planner while the chain CTAs need at most half of the SMs; forced
    here with HA_LA_TC_OVERLAP=2): the chain kernel runs next to the persistent prep kernel and takes each
    chunk as soon as its flag is published.  HA_LA_TC_OVERLAP=0 forces the sequential mode.  Same results in
    both, bit for bit, call after call."""
    if case.startswith("gdn"):
        w = synth.shrink(W["gdn_layer_4k"], seq_lens=[2048], hk=4, hv=4)
    elif case.startswith("kda"):
        w = synth.shrink(W["kda_8k"], seq_lens=[1000], hk=2, hv=4)
    else:
        w = synth.shrink(W["gdn_varlen"], seq_lens=[700, 0, 65, 1500], hk=2, hv=2)
    if case.endswith("nv64"):
        monkeypatch.setenv("HA_LA_TC_NV", "64")
    if case.endswith("nv128"):                           # the whole-head kernel (state in tensor memory)
        monkeypatch.setenv("HA_LA_TC_NV", "128")
    inp = synth.make_inputs(w, seed=37)
    monkeypatch.setenv("HA_LA_TC_OVERLAP", "0")
    o_seq, h_seq, st_seq = helpers.run_gpu(inp)
    monkeypatch.setenv("HA_LA_TC_OVERLAP", "2")
    o_con, h_con, st_con = helpers.run_gpu(inp)
    o_con2, h_con2, _ = helpers.run_gpu(inp)
    assert st_seq == 0 and st_con == 0
    np.testing.assert_array_equal(o_con, o_seq)
    np.testing.assert_array_equal(h_con, h_seq)
    np.testing.assert_array_equal(o_con2, o_seq)
    helpers.check_parity(inp)


def test_workspace_contents_do_not_matter(monkeypatch):
    """The workspace is scratch: whatever it holds on entry (small integers, all ones, an earlier call's
    flags) must not change the result -- in particular not pass for a 'chunk is ready' flag."""
    import torch
    import paper_2609_32114_b200 as ha

    monkeypatch.setenv("HA_LA_TC_OVERLAP", "2")          # concurrent mode whatever the planner would choose
    w = synth.shrink(W["gdn_layer_4k"], seq_lens=[1500], hk=2, hv=4)
    inp = synth.make_inputs(w, seed=41)
    d = helpers.to_device(inp)

    def call(ws=None):
        o, hT, st, ws_out = ha.ha_la_prefill(d["q"], d["k"], d["v"], d["g"], d["beta"], variant=w.variant, h0=d["h0"],
                                             cu_seqlens=d["cu_seqlens"], max_seqlen=d["max_seqlen"], workspace=ws)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        return o.clone(), hT.clone(), ws_out

    o0, h0, ws0 = call()
    for fill in (0x01, 0xFF, 0x00):
        ws = torch.full_like(ws0, fill)
        o1, h1, _ = call(ws)
        assert torch.equal(o1, o0) and torch.equal(h1, h0)
    ints = torch.arange(ws0.numel() // 4, dtype=torch.int32, device=ws0.device) % 64   # small counters everywhere
    o2, h2, _ = call(ints.view(torch.uint8))
    assert torch.equal(o2, o0) and torch.equal(h2, h0)
    o3, h3, _ = call(ws0)                                                                # an earlier call's workspace
    assert torch.equal(o3, o0) and torch.equal(h3, h0)


def test_back_to_back_calls_share_a_workspace(monkeypatch):
    """Many calls queued on one stream without synchronising in between, alternating between two problems
    of different shape that share one workspace (so every call sees the other's leftovers and the
    launch-mode switches between concurrent and sequential): results must equal the first call's."""
    import torch
    import paper_2609_32114_b200 as ha

    monkeypatch.setenv("HA_LA_TC_OVERLAP", "2")          # concurrent mode wherever the chain leaves SMs free
    wa = synth.shrink(W["gdn_layer_4k"], seq_lens=[1024], hk=2, hv=2)           # few chains: concurrent mode
    wb = synth.shrink(W["gdn_varlen"], seq_lens=[200, 0, 333, 64] * 10, hk=2, hv=4)   # 160 chains: sequential
    ia, ib = synth.make_inputs(wa, seed=43), synth.make_inputs(wb, seed=44)
    da, db = helpers.to_device(ia), helpers.to_device(ib)

    def call(d, w, ws):
        return ha.ha_la_prefill(d["q"], d["k"], d["v"], d["g"], d["beta"], variant=w.variant, h0=d["h0"],
                                cu_seqlens=d["cu_seqlens"], max_seqlen=d["max_seqlen"], workspace=ws)

    _, _, _, ws_a = call(da, wa, None)
    _, _, _, ws_b = call(db, wb, None)
    ws = ws_a if ws_a.numel() >= ws_b.numel() else ws_b
    ref_a = call(da, wa, ws)
    ref_b = call(db, wb, ws)
    torch.cuda.synchronize()
    ref_a = (ref_a[0].clone(), ref_a[1].clone())
    ref_b = (ref_b[0].clone(), ref_b[1].clone())
    outs = []
    for it in range(12):
        d, w = (da, wa) if it % 2 == 0 else (db, wb)
        o, hT, st, _ = call(d, w, ws)
        outs.append((o.clone(), hT.clone(), st))                 # clones are queued on the same stream, in order
    torch.cuda.synchronize()
    for it, (o, hT, st) in enumerate(outs):
        ref = ref_a if it % 2 == 0 else ref_b
        assert int(st.item()) == 0
        assert torch.equal(o, ref[0]) and torch.equal(hT, ref[1]), f"call {it} differs"
    helpers.check_parity(ia)
    helpers.check_parity(ib)


def test_two_streams_in_flight(monkeypatch):
    """Calls on two streams at once, each with its own workspace: the prep and chain kernels of the two
    calls compete for the SMs (together they want more than there are), nothing may deadlock or mix up."""
    import torch
    import paper_2609_32114_b200 as ha

    monkeypatch.setenv("HA_LA_TC_OVERLAP", "2")          # both calls in the concurrent mode
    w1 = synth.shrink(W["gdn_layer_4k"], seq_lens=[2048], hk=8, hv=8)
    w2 = synth.shrink(W["kda_8k"], seq_lens=[1024], hk=4, hv=8)
    i1, i2 = synth.make_inputs(w1, seed=51), synth.make_inputs(w2, seed=52)
    d1, d2 = helpers.to_device(i1), helpers.to_device(i2)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()

    def call(d, w, stream, ws=None):
        return ha.ha_la_prefill(d["q"], d["k"], d["v"], d["g"], d["beta"], variant=w.variant, h0=d["h0"],
                                cu_seqlens=d["cu_seqlens"], max_seqlen=d["max_seqlen"], workspace=ws,
                                stream=stream.cuda_stream)

    ref1 = call(d1, w1, s1)
    ref2 = call(d2, w2, s2)
    torch.cuda.synchronize()
    r1 = (ref1[0].clone(), ref1[1].clone()); r2 = (ref2[0].clone(), ref2[1].clone())
    ws1, ws2 = ref1[3], ref2[3]
    outs = []
    for it in range(6):
        a = call(d1, w1, s1, ws1)
        b = call(d2, w2, s2, ws2)
        with torch.cuda.stream(s1):
            oa = (a[0].clone(), a[1].clone(), a[2])
        with torch.cuda.stream(s2):
            ob = (b[0].clone(), b[1].clone(), b[2])
        outs.append((oa, ob))
    torch.cuda.synchronize()
    for oa, ob in outs:
        assert int(oa[2].item()) == 0 and int(ob[2].item()) == 0
        assert torch.equal(oa[0], r1[0]) and torch.equal(oa[1], r1[1])
        assert torch.equal(ob[0], r2[0]) and torch.equal(ob[1], r2[1])
    helpers.check_parity(i1)
    helpers.check_parity(i2)


@pytest.mark.parametrize("variant", ["gdn", "kda"])
def test_many_sequences_more_ctas_than_sms(variant):
    """A packed batch with many (sequence, V-head) chains of very different lengths: the chain kernel then
    has more CTAs than the GPU has SMs and starts them longest sequence first."""
    rng = np.random.default_rng(5)
    lens = [int(x) for x in rng.integers(1, 900, size=90)]
    lens[7] = 0
    lens[40] = 2500
    base = W["gdn_varlen"] if variant == "gdn" else W["kda_8k"]
    w = synth.shrink(base, seq_lens=lens, hk=2, hv=4, h0_std=0.02, varlen=True)
    inp = synth.make_inputs(w, seed=61)
    res = helpers.check_parity(inp, scale=0.5)
    print(variant, res)


def test_more_sequences_than_the_ranking_limit():
    """4,500 short sequences (0..130 tokens) in one packed batch: beyond 4,096 sequences the plan kernel leaves
    the launch order as given; the chain kernel then has thousands of CTAs, most of them with one or two chunks."""
    rng = np.random.default_rng(11)
    lens = [int(x) for x in rng.integers(0, 131, size=4500)]
    w = synth.shrink(W["gdn_varlen"], seq_lens=lens, hk=1, hv=1, h0_std=0.02, varlen=True)
    inp = synth.make_inputs(w, seed=67)
    pairs = [(n, 0) for n in sorted(set(range(0, 4500, 23)) | {1, 2, 4095, 4096, 4097, 4499, int(np.argmax(lens))})]
    res = helpers.check_parity(inp, pairs=pairs)
    print(res)


def test_randomized_shapes_widths_and_modes(monkeypatch):
    """Thirty seeded random cases: both variants, one to five sequences with lengths around the chunk
    boundaries (empty ones included), grouped heads, three gate strengths, with and without an initial state,
    every slice width of the chain kernel and every launch mode, against the oracle."""
    import random

    rng = random.Random(20260932114)
    for it in range(30):
        variant = rng.choice(["gdn", "kda"])
        lens = [rng.choice([0, 1, 63, 64, 65, 127, 128, 129, 200, 511, 700, 1000, 1537, 2048])
                for _ in range(rng.choice([1, 1, 2, 3, 5]))]
        if sum(lens) == 0:
            lens[0] = 77
        hk = rng.choice([1, 2, 4])
        hv = hk * rng.choice([1, 1, 2])
        base = W["gdn_varlen"] if variant == "gdn" else W["kda_8k"]
        w = synth.shrink(base, seq_lens=lens, hk=hk, hv=hv, gate_shift=rng.choice([-2.0, 0.0, 2.0]),
                         h0_std=rng.choice([0.0, 0.02]), varlen=True)
        inp = synth.make_inputs(w, seed=1000 + it)
        for var, val in (("HA_LA_TC_NV", rng.choice(["", "32", "64", "128"])),
                         ("HA_LA_TC_OVERLAP", rng.choice(["", "0", "2"]))):
            if val:
                monkeypatch.setenv(var, val)
            else:
                monkeypatch.delenv(var, raising=False)
        helpers.check_parity(inp, scale=rng.choice([1.0, 0.5]))
