"""Seeded synthetic inputs for delta-rule linear-attention prefill.

This module serves both the CUDA library's callers (tests, bench) and the CPU
oracle's tests.  It contains input preparation only (random draws, L2
normalisation, sigmoid / softplus activations, bf16 rounding) and none of the
method's arithmetic; it imports neither the CUDA binding nor the oracle.

The paper measures its kernels on synthetic shape sweeps (sequence length x
head count, FP16-class Q/K/V, FP32 gates and states, chunk 64) and end to end on
public QA / multimodal suites; none of those suites' items is reproduced here.
The five workloads below are shape stand-ins: the same tensor shapes, value
distributions and length mix, drawn from a counter-based generator.

Recipe (one Philox stream per workload, key = base seed + workload index, draws
in this fixed order, all in float32):
  1. sequence lengths (varlen only): integers uniform on [lo, hi] inclusive
  2. q, k ~ N(0,1), each (token, head) vector divided by its L2 norm
  3. v ~ N(0,1)
  4. beta = sigmoid(N(0,1))                     per (token, V-head)
  5. g = -softplus(N(0,1) + gate_shift)         per (token, V-head[, key channel])
  6. h0 ~ N(0, std 0.02)                        per (sequence, V-head), when used
q, k, v are then rounded to bf16 (round-to-nearest-even) for bf16 workloads and
kept as float32 arrays holding those rounded values; beta, g, h0 stay float32.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional, Sequence

import numpy as np

BASE_SEED = 2609032114


@dataclass(frozen=True)
class Workload:
    name: str
    variant: str                 # "gdn" | "kda"
    dtype: str                   # "bf16" | "fp32"  (dtype of q, k, v, o)
    hk: int
    hv: int
    dk: int
    dv: int
    seq_lens: Optional[Sequence[int]] = None   # fixed lengths; None = draw `num_seqs` lengths
    num_seqs: int = 1
    len_lo: int = 0
    len_hi: int = 0
    varlen: bool = False         # pass cu_seqlens (packed batch) instead of batch=1 / seqlen=T
    gate_shift: float = 0.0
    h0_std: float = 0.0          # 0 => no initial state (NULL)
    index: int = 0               # stream selector


# The five benchmark workloads.
WORKLOADS = {
    "gdn_fp32_small": Workload("gdn_fp32_small", "gdn", "fp32", 1, 1, 64, 64, seq_lens=(256,), index=0),
    "gdn_layer_4k": Workload("gdn_layer_4k", "gdn", "bf16", 16, 16, 128, 128, seq_lens=(4096,),
                             gate_shift=2.0, index=1),
    "gdn_gva_16k": Workload("gdn_gva_16k", "gdn", "bf16", 16, 32, 128, 128, seq_lens=(16384,),
                            gate_shift=2.0, h0_std=0.02, index=2),
    "kda_8k": Workload("kda_8k", "kda", "bf16", 32, 32, 128, 128, seq_lens=(8192,), gate_shift=2.0, index=3),
    "gdn_varlen": Workload("gdn_varlen", "gdn", "bf16", 16, 16, 128, 128, seq_lens=None, num_seqs=8,
                           len_lo=512, len_hi=32768, varlen=True, gate_shift=2.0, h0_std=0.02, index=4),
}


def shrink(w: Workload, *, seq_lens=None, hk=None, hv=None, **kw) -> Workload:
    """A smaller case of the same workload (same distributions and stream)."""
    upd = dict(kw)
    if seq_lens is not None:
        upd.update(seq_lens=tuple(int(x) for x in seq_lens), num_seqs=len(seq_lens))
    if hk is not None:
        upd["hk"] = hk
    if hv is not None:
        upd["hv"] = hv
    return replace(w, **upd)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> nearest bf16 (ties to even), returned as float32 holding the rounded value."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16) << 16
    return r.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 array holding bf16-representable values -> uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16).reshape(x.shape)


def _softplus(x):
    return np.logaddexp(np.float32(0), x).astype(np.float32)


def _normal_chunks(rng, shape):
    out = np.empty(shape, dtype=np.float32)
    flat = out.reshape(-1)
    step = 1 << 24
    for s in range(0, flat.size, step):
        e = min(s + step, flat.size)
        flat[s:e] = rng.standard_normal(e - s, dtype=np.float32)
    return out


def make_inputs(w: Workload, seed: int = BASE_SEED) -> dict:
    """Draw one batch for workload `w`.  Returns numpy arrays:

    q, k [T, HK, dk]; v [T, HV, dv]; beta [T, HV]; g [T, HV] (gdn) or [T, HV, dk] (kda);
    h0 [N, HV, dk, dv] or None; cu_seqlens int32 [N+1]; seq_lens (list); plus the workload.
    """
    rng = np.random.Generator(np.random.Philox(key=int(seed) + int(w.index)))
    if w.seq_lens is None:
        lens = [int(x) for x in rng.integers(w.len_lo, w.len_hi + 1, size=w.num_seqs)]
    else:
        lens = [int(x) for x in w.seq_lens]
    N = len(lens)
    cu = np.zeros(N + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    T = int(cu[-1])

    def unit(shape):
        x = _normal_chunks(rng, shape)
        n = np.sqrt(np.sum(x.astype(np.float32) ** 2, axis=-1, keepdims=True, dtype=np.float32))
        return (x / np.maximum(n, np.float32(1e-20))).astype(np.float32)

    q = unit((T, w.hk, w.dk))
    k = unit((T, w.hk, w.dk))
    v = _normal_chunks(rng, (T, w.hv, w.dv))
    bl = _normal_chunks(rng, (T, w.hv))
    beta = (np.float32(1) / (np.float32(1) + np.exp(-bl))).astype(np.float32)
    gshape = (T, w.hv) if w.variant == "gdn" else (T, w.hv, w.dk)
    g = (-_softplus(_normal_chunks(rng, gshape) + np.float32(w.gate_shift))).astype(np.float32)
    h0 = None
    if w.h0_std > 0:
        h0 = (_normal_chunks(rng, (N, w.hv, w.dk, w.dv)) * np.float32(w.h0_std)).astype(np.float32)
    if w.dtype == "bf16":
        q, k, v = round_to_bf16(q), round_to_bf16(k), round_to_bf16(v)
    return dict(workload=w, q=q, k=k, v=v, beta=beta, g=g, h0=h0, cu_seqlens=cu, seq_lens=lens, T=T, N=N)


# ---- work model (per token of one V-head, chunk C): used by the bench and checked in the tests ----

def macs_per_chunk_head(C: int, d: int) -> float:
    """Matrix MACs of the six chunkwise operators for one (chunk, head): 5 C^2 d + 3 C d^2 + C^3/2.

    This is the count that reproduces the paper's Table 1 "MACs" column for the
    linear-attention layer (H=16, d=128, C=64): 0.75 / 1.51 / 3.02 / 6.04 GMAC at
    512 / 1k / 2k / 4k tokens.
    """
    return 5.0 * C * C * d + 3.0 * C * d * d + C ** 3 / 2.0


def algorithmic_flops(w: Workload, total_tokens: int, C: int = 64) -> float:
    """2 x MACs; with grouped values the raw K K^T / Q K^T products count once per QK head."""
    d = w.dk
    per_tok_v = 2.0 * (3.0 * C * d + 3.0 * d * d + C * C / 2.0)
    per_tok_qk = 2.0 * (2.0 * C * d)
    return total_tokens * (w.hv * per_tok_v + w.hk * per_tok_qk)


def algorithmic_bytes(w: Workload, total_tokens: int, num_seqs: int, with_hT: bool = True) -> float:
    """Bytes the method must touch once: q,k,v in, o out, g, beta, h0 in (if any), hT out."""
    e = 2 if w.dtype == "bf16" else 4
    per_tok = 2 * w.hk * w.dk * e + 2 * w.hv * w.dv * e + w.hv * 4
    per_tok += w.hv * 4 * (w.dk if w.variant == "kda" else 1)
    state = num_seqs * w.hv * w.dk * w.dv * 4
    return total_tokens * per_tok + (state if w.h0_std > 0 else 0) + (state if with_hT else 0)
