"""GPU parity of the decoding step (ha_la_decode): one new token per sequence against the fp64 oracle, which
evaluates the same recurrence on sequences of length one with the state as h0."""
import numpy as np
import pytest

from paper_2609_32114_b200 import synth
from tests import helpers

pytestmark = pytest.mark.gpu
W = synth.WORKLOADS


def _inputs(variant, dtype, d, n, hk, hv, seed, state_std=0.5):
    base = W["gdn_varlen"] if variant == "gdn" else W["kda_8k"]
    w = synth.shrink(base, seq_lens=[1] * n, hk=hk, hv=hv, dtype=dtype, dk=d, dv=d, h0_std=state_std, varlen=True,
                     gate_shift=0.0)
    return synth.make_inputs(w, seed=seed)


def _run(inp, scale=1.0, state=True, inplace=True):
    import torch
    import paper_2609_32114_b200 as ha

    w = inp["workload"]
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    dev = lambda a, t: torch.from_numpy(np.ascontiguousarray(a)).cuda().to(t).contiguous()
    q, k, v = dev(inp["q"], dt), dev(inp["k"], dt), dev(inp["v"], dt)
    g, beta = dev(inp["g"], torch.float32), dev(inp["beta"], torch.float32)
    st = dev(inp["h0"], torch.float32) if state else None
    out = None if inplace or st is None else torch.empty_like(st)
    o, new = ha.ha_la_decode(q, k, v, g, beta, st, variant=w.variant, scale=scale, state_out=out)
    torch.cuda.synchronize()
    return o.float().cpu().numpy(), new.cpu().numpy().astype(np.float64), (st.cpu().numpy() if st is not None else None)


def _check(inp, o, new_state, scale=1.0, state=True):
    import oracle

    w = inp["workload"]
    o_ref, h_ref, _ = oracle.recurrent(inp["q"], inp["k"], inp["v"], inp["g"], inp["beta"], variant=w.variant,
                                       h0=inp["h0"] if state else None, cu_seqlens=inp["cu_seqlens"], scale=scale)
    tol = helpers.TOL[w.dtype]
    assert helpers.rel_max_err(o, o_ref) <= tol
    assert helpers.rel_max_err(new_state, h_ref) <= 1e-5       # the state is fp32 end to end in both dtypes


@pytest.mark.parametrize("variant", ["gdn", "kda"])
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("d", [64, 128])
def test_decode_step_matches_oracle(variant, dtype, d):
    inp = _inputs(variant, dtype, d, n=37, hk=2, hv=4, seed=71)
    o, new, _ = _run(inp, scale=0.7)
    _check(inp, o, new, scale=0.7)


def test_decode_without_state_and_out_of_place():
    inp = _inputs("gdn", "bf16", 128, n=5, hk=3, hv=3, seed=72)
    o, new, _ = _run(inp, state=False)
    _check(inp, o, new, state=False)
    o1, new1, st_after = _run(inp, inplace=False)
    o2, new2, _ = _run(inp, inplace=True)
    np.testing.assert_array_equal(o1, o2)
    np.testing.assert_array_equal(new1, new2)
    np.testing.assert_array_equal(st_after, inp["h0"])            # the input state was left alone
    _check(inp, o1, new1)


def test_empty_batch_is_a_no_op():
    import torch
    import paper_2609_32114_b200 as ha

    z = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt, device="cuda")
    o, new = ha.ha_la_decode(z(0, 2, 128), z(0, 2, 128), z(0, 2, 128), z(0, 2, dt=torch.float32),
                             z(0, 2, dt=torch.float32), z(0, 2, 128, 128, dt=torch.float32))
    torch.cuda.synchronize()
    assert o.shape[0] == 0 and new.shape[0] == 0


def test_prefill_then_decode_equals_one_long_prefill():
    """Prefill T tokens, then three decoding steps on the state it returned: the outputs and the final state equal
    those of the oracle run over all T + 3 tokens (only the state crosses the boundary)."""
    import torch
    import oracle
    import paper_2609_32114_b200 as ha

    T, extra = 200, 3
    w = synth.shrink(W["gdn_layer_4k"], seq_lens=[T + extra], hk=2, hv=4)
    inp = synth.make_inputs(w, seed=73)
    o_ref, h_ref, _ = oracle.recurrent(inp["q"], inp["k"], inp["v"], inp["g"], inp["beta"], variant="gdn")
    dev = lambda a, t: torch.from_numpy(np.ascontiguousarray(a)).cuda().to(t).contiguous()
    bf, f32 = torch.bfloat16, torch.float32
    q, k, v = dev(inp["q"], bf), dev(inp["k"], bf), dev(inp["v"], bf)
    g, beta = dev(inp["g"], f32), dev(inp["beta"], f32)
    o, hT, st, _ = ha.ha_la_prefill(q[None, :T], k[None, :T], v[None, :T], g[None, :T], beta[None, :T], variant="gdn")
    state = hT                                                     # [1, HV, d, d]
    outs = [o.reshape(T, 4, 128).float()]
    for t in range(T, T + extra):
        ot, state = ha.ha_la_decode(q[t:t + 1].contiguous(), k[t:t + 1].contiguous(), v[t:t + 1].contiguous(),
                                    g[t:t + 1].contiguous(), beta[t:t + 1].contiguous(), state, variant="gdn")
        outs.append(ot.float())
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    o_all = torch.cat(outs).cpu().numpy()
    assert helpers.rel_max_err(o_all, o_ref) <= helpers.TOL["bf16"]
    assert helpers.rel_max_err(state.cpu().numpy().astype(np.float64), h_ref) <= helpers.TOL["bf16"]
