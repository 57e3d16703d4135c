"""Pins for the CPU fp64 oracle: what the paper and the mathematics fix, not the oracle itself.

Each test is chosen so that a plausible slip in the oracle (dropped term, wrong
sign, transposed state, decay/erase order, pre- vs post-update output, head
mapping) fails at least one of them.
"""
import json
import os

import numpy as np
import pytest

import oracle
from oracle.chunked import chunked


def _rand(rng, T, HK, HV, dk, dv, variant, unit_keys=True, gate_scale=1.0):
    q = rng.standard_normal((T, HK, dk))
    k = rng.standard_normal((T, HK, dk))
    if unit_keys:
        q /= np.linalg.norm(q, axis=-1, keepdims=True)
        k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = rng.standard_normal((T, HV, dv))
    beta = 1.0 / (1.0 + np.exp(-rng.standard_normal((T, HV))))
    gs = (T, HV) if variant == "gdn" else (T, HV, dk)
    g = -np.logaddexp(0.0, rng.standard_normal(gs)) * gate_scale
    f = lambda a: a.astype(np.float32)
    return f(q), f(k), f(v), f(g), f(beta)


def _d(x):
    return np.asarray(x, dtype=np.float64)


# ---------------------------------------------------------------- worked examples (golden)

def test_worked_examples(golden_dir):
    with open(os.path.join(golden_dir, "worked_examples.json")) as f:
        cases = json.load(f)["cases"]
    assert len(cases) == 3
    for c in cases:
        q = np.array(c["q"], dtype=np.float32)[:, None, :]
        k = np.array(c["k"], dtype=np.float32)[:, None, :]
        v = np.array(c["v"], dtype=np.float32)[:, None, :]
        beta = np.array(c["beta"], dtype=np.float32)[:, None]
        g = np.log(np.array(c["alpha"], dtype=np.float64)).astype(np.float32)
        g = g[:, None] if c["variant"] == "gdn" else g[:, None, :]
        h0 = None if c["h0"] is None else np.array(c["h0"], dtype=np.float32)[None, None]
        o, hT, _ = oracle.recurrent(q, k, v, g, beta, variant=c["variant"], h0=h0)
        # g went through float32 (log 0.5 is not exact), hence 1e-6 rather than 1e-12
        np.testing.assert_allclose(o[:, 0, :], np.array(c["o"]), rtol=0, atol=1e-6, err_msg=c["name"])
        np.testing.assert_allclose(hT[0, 0], np.array(c["hT"]), rtol=0, atol=1e-6, err_msg=c["name"])
        o2, hT2 = chunked(q, k, v, g, beta, variant=c["variant"], h0=h0, chunk=64)
        np.testing.assert_allclose(o2[:, 0, :], np.array(c["o"]), rtol=0, atol=1e-6)
        np.testing.assert_allclose(hT2[0, 0], np.array(c["hT"]), rtol=0, atol=1e-6)


# ---------------------------------------------------------------- single token closed form (I1)

@pytest.mark.parametrize("variant", ["gdn", "kda"])
def test_single_token_closed_form(variant):
    rng = np.random.default_rng(1)
    dk, dv = 5, 3
    q, k, v, g, beta = _rand(rng, 1, 1, 1, dk, dv, variant, unit_keys=False)
    h0 = rng.standard_normal((1, 1, dk, dv)).astype(np.float32)
    scale = 0.7
    o, hT, _ = oracle.recurrent(q, k, v, g, beta, variant=variant, h0=h0, scale=scale)
    q1, k1, v1, b1 = _d(q[0, 0]), _d(k[0, 0]), _d(v[0, 0]), float(beta[0, 0])
    D = np.exp(_d(g[0, 0])) * np.eye(dk) if variant == "gdn" else np.diag(np.exp(_d(g[0, 0])))
    kq = float(k1 @ q1)
    expect = scale * (_d(h0[0, 0]).T @ D @ (q1 - b1 * kq * k1) + b1 * kq * v1)
    np.testing.assert_allclose(o[0, 0], expect, rtol=1e-12, atol=1e-13)
    # zero initial state: o_1 = scale * beta (k.q) v
    o0, _, _ = oracle.recurrent(q, k, v, g, beta, variant=variant, scale=scale)
    np.testing.assert_allclose(o0[0, 0], scale * b1 * kq * v1, rtol=1e-12, atol=1e-13)
    assert abs(kq) > 1e-3 and np.abs(o0).max() > 0     # the output uses the UPDATED state


@pytest.mark.parametrize("variant", ["gdn", "kda"])
def test_decode_step_closed_form_batched(variant):
    """The decoding step is the recurrence on sequences of length one with the state as h0: a packed batch of
    N such sequences (grouped values, HV = 2 HK) equals the single-token closed form per (sequence, V-head),
    and the new state equals decay(h0) + beta k (v - decay(h0)^T k)^T written out."""
    rng = np.random.default_rng(11)
    N, hk, hv, dk, dv = 5, 2, 4, 6, 6
    q, k, v, g, beta = _rand(rng, N, hk, hv, dk, dv, variant, unit_keys=False)
    h0 = rng.standard_normal((N, hv, dk, dv)).astype(np.float32)
    cu = np.arange(N + 1, dtype=np.int32)
    o, hT, _ = oracle.recurrent(q, k, v, g, beta, variant=variant, h0=h0, cu_seqlens=cu, scale=1.3)
    for n in range(N):
        for j in range(hv):
            jq = j // (hv // hk)
            qq, kk, vv, b = _d(q[n, jq]), _d(k[n, jq]), _d(v[n, j]), float(beta[n, j])
            dec = np.exp(_d(g[n, j])) * np.ones(dk)
            hd = dec[:, None] * _d(h0[n, j])
            hnew = hd + b * np.outer(kk, vv - hd.T @ kk)
            np.testing.assert_allclose(hT[n, j], hnew, rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(o[n, j], 1.3 * (hnew.T @ qq), rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- matrix form of the recurrence

@pytest.mark.parametrize("variant", ["gdn", "kda"])
def test_matrix_form_small(variant):
    """S_t = S_{t-1} Diag(alpha_t) (I - beta k k^T) + beta v k^T, o_t = S_t q_t, by explicit matrices."""
    rng = np.random.default_rng(2)
    T, dk, dv = 7, 4, 3
    q, k, v, g, beta = _rand(rng, T, 1, 1, dk, dv, variant)
    h0 = rng.standard_normal((1, 1, dk, dv)).astype(np.float32)
    S = _d(h0[0, 0]).T.copy()                     # d_v x d_k
    outs = []
    for t in range(T):
        al = np.exp(_d(g[t, 0]))
        Dm = al * np.eye(dk) if variant == "gdn" else np.diag(al)
        kt = _d(k[t, 0])[:, None]
        S = S @ Dm @ (np.eye(dk) - beta[t, 0] * (kt @ kt.T)) + float(beta[t, 0]) * _d(v[t, 0])[:, None] @ kt.T
        outs.append(S @ _d(q[t, 0]))
    o, hT, _ = oracle.recurrent(q, k, v, g, beta, variant=variant, h0=h0)
    np.testing.assert_allclose(o[:, 0], np.array(outs), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(hT[0, 0], S.T, rtol=1e-11, atol=1e-12)   # hT is d_k x d_v = S^T


# ---------------------------------------------------------------- chunked == recurrent (I2)

@pytest.mark.parametrize("variant", ["gdn", "kda"])
@pytest.mark.parametrize("C", [4, 16, 64])
@pytest.mark.parametrize("T", [1, 7, 13, 16])
def test_chunked_equals_recurrent_tiny(variant, C, T):
    rng = np.random.default_rng(100 + T + C)
    q, k, v, g, beta = _rand(rng, T, 1, 1, 6, 5, variant)
    h0 = rng.standard_normal((1, 1, 6, 5)).astype(np.float32)
    o, hT, _ = oracle.recurrent(q, k, v, g, beta, variant=variant, h0=h0, scale=0.5)
    o2, hT2 = chunked(q, k, v, g, beta, variant=variant, h0=h0, scale=0.5, chunk=C)
    np.testing.assert_allclose(o2, o, rtol=0, atol=1e-12)
    np.testing.assert_allclose(hT2, hT, rtol=0, atol=1e-12)


@pytest.mark.parametrize("variant", ["gdn", "kda"])
def test_chunked_equals_recurrent_varlen_gva(variant):
    rng = np.random.default_rng(7)
    lens = [70, 0, 129, 64, 5]
    cu = np.concatenate([[0], np.cumsum(lens)])
    T = int(cu[-1])
    q, k, v, g, beta = _rand(rng, T, 2, 4, 16, 8, variant)
    h0 = (0.1 * rng.standard_normal((len(lens), 4, 16, 8))).astype(np.float32)
    o, hT, _ = oracle.recurrent(q, k, v, g, beta, variant=variant, h0=h0, cu_seqlens=cu)
    o2, hT2 = chunked(q, k, v, g, beta, variant=variant, h0=h0, cu_seqlens=cu, chunk=64)
    np.testing.assert_allclose(o2, o, rtol=0, atol=1e-11)
    np.testing.assert_allclose(hT2, hT, rtol=0, atol=1e-11)
    np.testing.assert_allclose(hT[1], _d(h0[1]), rtol=0, atol=0)       # empty sequence: hT = h0


# ---------------------------------------------------------------- beta = 0 freezes the state (I3a)

@pytest.mark.parametrize("variant", ["gdn", "kda"])
def test_beta_zero_frozen_state(variant):
    rng = np.random.default_rng(3)
    T, dk, dv = 9, 4, 3
    q, k, v, g, beta = _rand(rng, T, 1, 1, dk, dv, variant)
    beta[:] = 0
    h0 = rng.standard_normal((1, 1, dk, dv)).astype(np.float32)
    o, hT, _ = oracle.recurrent(q, k, v, g, beta, variant=variant, h0=h0, scale=2.0)
    G = np.cumsum(_d(g[:, 0]), axis=0)
    for t in range(T):
        dec = np.exp(G[t]) * np.ones(dk)
        np.testing.assert_allclose(o[t, 0], 2.0 * (_d(h0[0, 0]) * dec[:, None]).T @ _d(q[t, 0]), atol=1e-13)
    np.testing.assert_allclose(hT[0, 0], _d(h0[0, 0]) * (np.exp(G[-1]) * np.ones(dk))[:, None], atol=1e-13)


# ---------------------------------------------------------------- small beta -> causal prefix sum (I3b)

def test_small_beta_is_linear_attention():
    rng = np.random.default_rng(4)
    T, dk, dv = 12, 4, 3
    q, k, v, g, beta = _rand(rng, T, 1, 1, dk, dv, "gdn")
    g[:] = 0
    eps = 1e-7
    beta[:] = eps
    o, _, _ = oracle.recurrent(q, k, v, g, beta)
    kv = np.cumsum(_d(k[:, 0])[:, :, None] * _d(v[:, 0])[:, None, :], axis=0)    # prefix sum of k v^T
    expect = np.einsum("tc,tcx->tx", _d(q[:, 0]), kv)
    b = float(np.float32(eps))
    np.testing.assert_allclose(o[:, 0] / b, expect, rtol=0, atol=1e-5)


# ---------------------------------------------------------------- orthogonal keys (I3c)

@pytest.mark.parametrize("variant", ["gdn"])
def test_orthogonal_keys_closed_form(variant):
    rng = np.random.default_rng(5)
    T = dk = 6
    dv = 4
    Q_, _ = np.linalg.qr(rng.standard_normal((dk, dk)))
    q, k, v, g, beta = _rand(rng, T, 1, 1, dk, dv, variant)
    k[:, 0, :] = Q_.astype(np.float32)              # rows orthonormal up to float32 rounding
    o, hT, _ = oracle.recurrent(q, k, v, g, beta, scale=1.5)
    G = np.cumsum(_d(g[:, 0]))
    kk = _d(k[:, 0])
    for t in range(T):
        acc = np.zeros(dv)
        for j in range(t + 1):
            acc += np.exp(G[t] - G[j]) * beta[j, 0] * float(kk[j] @ _d(q[t, 0])) * _d(v[j, 0])
        np.testing.assert_allclose(o[t, 0], 1.5 * acc, rtol=0, atol=2e-6)   # orthogonality holds to fp32 only
    # alpha = 1, beta = 1, orthonormal keys: the state is exactly sum_j k_j v_j^T
    g[:] = 0
    beta[:] = 1
    _, hT, _ = oracle.recurrent(q, k, v, g, beta)
    np.testing.assert_allclose(hT[0, 0], kk.T @ _d(v[:, 0]), rtol=0, atol=2e-6)


# ---------------------------------------------------------------- retrieval identity (I4)

@pytest.mark.parametrize("variant", ["gdn", "kda"])
def test_retrieval_identity(variant):
    """Unit-norm keys, beta = 1, q = k  =>  o_t = v_t for any gates (decay first, then erase+write)."""
    rng = np.random.default_rng(6)
    T, dk, dv = 20, 8, 5
    q, k, v, g, beta = _rand(rng, T, 1, 1, dk, dv, variant)
    kd = _d(k)
    kd /= np.linalg.norm(kd, axis=-1, keepdims=True)
    k = kd.astype(np.float32)
    beta[:] = 1
    h0 = rng.standard_normal((1, 1, dk, dv)).astype(np.float32)
    o, _, _ = oracle.recurrent(k, k, v, g, beta, variant=variant, h0=h0)
    np.testing.assert_allclose(o[:, 0], _d(v[:, 0]), rtol=0, atol=5e-6)     # |k| = 1 to fp32 only
    # general beta: S_t k_t = (1 - beta)(decayed S_{t-1}) k_t + beta v_t  -- checked on the last token
    q2, k2, v2, g2, b2 = _rand(rng, 3, 1, 1, dk, dv, variant)
    o3, hT3, _ = oracle.recurrent(k2, k2, v2, g2, b2, variant=variant)
    _, hT2, _ = oracle.recurrent(k2[:2], k2[:2], v2[:2], g2[:2], b2[:2], variant=variant)
    dec = np.exp(_d(g2[2, 0])) * np.ones(dk)
    kt = _d(k2[2, 0])
    nk = float(kt @ kt)
    pred = (hT2[0, 0] * dec[:, None]).T @ kt
    expect = pred + float(b2[2, 0]) * nk * (_d(v2[2, 0]) - pred)
    np.testing.assert_allclose(o3[2, 0], expect, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- independence (I5)

@pytest.mark.parametrize("variant", ["gdn", "kda"])
def test_independence_heads_sequences_gva_columns(variant):
    rng = np.random.default_rng(8)
    lens = [11, 3, 18]
    cu = np.concatenate([[0], np.cumsum(lens)])
    T, HK, HV, dk, dv = int(cu[-1]), 2, 4, 6, 4
    q, k, v, g, beta = _rand(rng, T, HK, HV, dk, dv, variant)
    h0 = rng.standard_normal((3, HV, dk, dv)).astype(np.float32)
    o, hT, _ = oracle.recurrent(q, k, v, g, beta, variant=variant, h0=h0, cu_seqlens=cu)
    # (a) packed batch == one call per sequence
    for n in range(3):
        s, e = cu[n], cu[n + 1]
        on, hTn, _ = oracle.recurrent(q[s:e], k[s:e], v[s:e], g[s:e], beta[s:e], variant=variant, h0=h0[n:n + 1])
        np.testing.assert_array_equal(on, o[s:e])
        np.testing.assert_array_equal(hTn[0], hT[n])
    # (b) grouped values == explicitly repeated q, k (V-head j reads QK-head j // 2)
    qe, ke = np.repeat(q, 2, axis=1), np.repeat(k, 2, axis=1)
    oe, hTe, _ = oracle.recurrent(qe, ke, v, g, beta, variant=variant, h0=h0, cu_seqlens=cu)
    np.testing.assert_array_equal(oe, o)
    np.testing.assert_array_equal(hTe, hT)
    assert not np.array_equal(q[:, 0], q[:, 1])
    # (c) each V-head on its own
    for j in range(HV):
        jq = j // 2
        oj, hTj, _ = oracle.recurrent(q[:, jq:jq + 1], k[:, jq:jq + 1], v[:, j:j + 1], g[:, j:j + 1],
                                      beta[:, j:j + 1], variant=variant, h0=h0[:, j:j + 1], cu_seqlens=cu)
        np.testing.assert_array_equal(oj[:, 0], o[:, j])
        np.testing.assert_array_equal(hTj[:, 0], hT[:, j])
    # (d) a column block of o / hT depends only on the same columns of v / h0
    oc, hTc, _ = oracle.recurrent(q, k, v[:, :, 1:3], g, beta, variant=variant, h0=h0[..., 1:3], cu_seqlens=cu)
    np.testing.assert_array_equal(oc, o[:, :, 1:3])
    np.testing.assert_array_equal(hTc, hT[..., 1:3])
    # (e) the `pairs` selector computes exactly the selected (sequence, head) and nothing else
    op, hTp, _ = oracle.recurrent(q, k, v, g, beta, variant=variant, h0=h0, cu_seqlens=cu, pairs=[(2, 1), (0, 3)])
    np.testing.assert_array_equal(op[cu[2]:cu[3], 1], o[cu[2]:cu[3], 1])
    np.testing.assert_array_equal(op[cu[0]:cu[1], 3], o[cu[0]:cu[1], 3])
    np.testing.assert_array_equal(hTp[2, 1], hT[2, 1])
    assert np.all(op[cu[1]:cu[2]] == 0) and np.all(op[:, 0] == 0)


# ---------------------------------------------------------------- split / resume (I6)

@pytest.mark.parametrize("variant", ["gdn", "kda"])
@pytest.mark.parametrize("T1", [1, 64, 70])
def test_split_resume(variant, T1):
    rng = np.random.default_rng(9)
    T, dk, dv = 150, 8, 6          # d_k != d_v: a transposed hT would not even have the right shape
    q, k, v, g, beta = _rand(rng, T, 1, 2, dk, dv, variant)
    o, hT, _ = oracle.recurrent(q, k, v, g, beta, variant=variant)
    oa, ha, _ = oracle.recurrent(q[:T1], k[:T1], v[:T1], g[:T1], beta[:T1], variant=variant)
    ob, hb, _ = oracle.recurrent(q[T1:], k[T1:], v[T1:], g[T1:], beta[T1:], variant=variant,
                                 h0=ha.astype(np.float32))
    # the carried state passes through float32 here, hence 1e-6
    np.testing.assert_allclose(np.concatenate([oa, ob]), o, rtol=0, atol=1e-6)
    np.testing.assert_allclose(hb, hT, rtol=0, atol=1e-6)


# ---------------------------------------------------------------- linearity (I7)

@pytest.mark.parametrize("variant", ["gdn", "kda"])
def test_linearity(variant):
    rng = np.random.default_rng(10)
    T, dk, dv = 10, 5, 4
    q, k, v, g, beta = _rand(rng, T, 1, 1, dk, dv, variant)
    o1, h1, _ = oracle.recurrent(q, k, v, g, beta, variant=variant, scale=1.0)
    o3, h3, _ = oracle.recurrent(q, k, v, g, beta, variant=variant, scale=3.0)
    np.testing.assert_allclose(o3, 3.0 * o1, rtol=1e-13)
    np.testing.assert_array_equal(h3, h1)
    o2v, h2v, _ = oracle.recurrent(q, k, 2 * v, g, beta, variant=variant)          # exact in fp32
    np.testing.assert_allclose(o2v, 2 * o1, rtol=1e-13)
    np.testing.assert_allclose(h2v, 2 * h1, rtol=1e-13)
    q2 = rng.standard_normal(q.shape).astype(np.float32)
    _, hq, _ = oracle.recurrent(q2, k, v, g, beta, variant=variant)
    np.testing.assert_array_equal(hq, h1)                                           # hT does not depend on q


# ---------------------------------------------------------------- boundedness (I8)

@pytest.mark.parametrize("variant", ["gdn", "kda"])
def test_state_bounded_with_unit_keys(variant):
    rng = np.random.default_rng(11)
    T, dk, dv = 300, 16, 8
    q, k, v, g, beta = _rand(rng, T, 1, 1, dk, dv, variant, gate_scale=0.05)
    kd = _d(k); kd /= np.linalg.norm(kd, axis=-1, keepdims=True)
    k = (kd * (1 - 1e-6)).astype(np.float32)        # |k| <= 1 after rounding
    h0 = rng.standard_normal((1, 1, dk, dv)).astype(np.float32)
    bound = np.linalg.norm(_d(h0[0, 0]))
    for t in (1, 50, 300):
        _, hT, _ = oracle.recurrent(q[:t], k[:t], v[:t], g[:t], beta[:t], variant=variant, h0=h0)
        b = bound + np.sum(_d(beta[:t, 0]) * np.linalg.norm(_d(v[:t, 0]), axis=-1))
        assert np.linalg.norm(hT[0, 0]) <= b * (1 + 1e-9)
    assert np.isfinite(hT).all()


# ---------------------------------------------------------------- argument checking

def test_oracle_rejects_bad_pairs():
    rng = np.random.default_rng(12)
    q, k, v, g, beta = _rand(rng, 4, 1, 1, 4, 4, "gdn")
    with pytest.raises(RuntimeError):
        oracle.recurrent(q, k, v, g, beta, pairs=[(0, 5)])
