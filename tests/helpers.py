"""Shared helpers of the GPU parity tests: run the CUDA library and the CPU oracle on the same
seeded inputs and compare with the stated error metric (max-norm relative error per output tensor)."""
import numpy as np

TOL = {"bf16": 2e-2, "fp32": 1e-4}     # max|err| / max|ref|, per output tensor (the stated tolerances)


def to_device(inp, device="cuda"):
    import torch

    w = inp["workload"]
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    T = inp["T"]

    def dev(a, dtype):
        return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(device).to(dtype).contiguous()

    d = dict(q=dev(inp["q"], dt), k=dev(inp["k"], dt), v=dev(inp["v"], dt), g=dev(inp["g"], torch.float32),
             beta=dev(inp["beta"], torch.float32), h0=dev(inp["h0"], torch.float32))
    if w.varlen:
        d["cu_seqlens"] = torch.from_numpy(inp["cu_seqlens"].astype(np.int32)).to(device)
        d["max_seqlen"] = max(inp["seq_lens"]) if inp["seq_lens"] else 0
    else:
        # equal-length rows: [B, T_row, ...]
        B = inp["N"]
        for key in ("q", "k", "v", "g", "beta"):
            t = d[key]
            d[key] = t.reshape(B, T // B, *t.shape[1:]).contiguous()
        d["cu_seqlens"] = None
        d["max_seqlen"] = 0
    return d


def run_gpu(inp, scale=1.0, **kw):
    """Calls the library through its C ABI (via the ctypes binding).  Returns numpy o [T,HV,dv], hT, status."""
    import torch
    import paper_2609_32114_b200 as ha

    w = inp["workload"]
    d = to_device(inp)
    o, hT, status, _ = ha.ha_la_prefill(d["q"], d["k"], d["v"], d["g"], d["beta"], variant=w.variant, h0=d["h0"],
                                        cu_seqlens=d["cu_seqlens"], max_seqlen=d["max_seqlen"], scale=scale, **kw)
    torch.cuda.synchronize()
    o = o.float().cpu().numpy().reshape(inp["T"], w.hv, w.dv)
    return o, hT.cpu().numpy().astype(np.float64), int(status.item())


def run_oracle(inp, scale=1.0, pairs=None):
    import oracle

    w = inp["workload"]
    o, hT, _ = oracle.recurrent(inp["q"], inp["k"], inp["v"], inp["g"], inp["beta"], variant=w.variant,
                                h0=inp["h0"], cu_seqlens=inp["cu_seqlens"], scale=scale, pairs=pairs)
    return o, hT


def rel_max_err(x, ref):
    m = float(np.max(np.abs(ref))) if ref.size else 0.0
    e = float(np.max(np.abs(np.asarray(x, dtype=np.float64) - ref))) if ref.size else 0.0
    return e / m if m > 0 else e


def nmse(x, ref):
    den = float(np.sum(ref * ref))
    return float(np.sum((np.asarray(x, dtype=np.float64) - ref) ** 2)) / den if den > 0 else 0.0


def check_parity(inp, scale=1.0, pairs=None, tol=None, **kw):
    """GPU vs oracle on all (or the selected) (sequence, V-head) pairs.  Returns the error figures."""
    w = inp["workload"]
    tol = TOL[w.dtype] if tol is None else tol
    o, hT, status = run_gpu(inp, scale=scale, **kw)
    assert status == 0, f"device status word = {status}"
    assert np.isfinite(o).all() and np.isfinite(hT).all()
    o_ref, hT_ref = run_oracle(inp, scale=scale, pairs=pairs)
    if pairs is not None:
        cu = inp["cu_seqlens"]
        rows = []
        for (n, j) in pairs:
            rows.append((slice(int(cu[n]), int(cu[n + 1])), j))
        o_sel = np.concatenate([o[r, j].ravel() for r, j in rows]) if rows else np.zeros(0)
        o_ref_sel = np.concatenate([o_ref[r, j].ravel() for r, j in rows]) if rows else np.zeros(0)
        h_sel = np.stack([hT[n, j] for n, j in pairs])
        h_ref_sel = np.stack([hT_ref[n, j] for n, j in pairs])
    else:
        o_sel, o_ref_sel, h_sel, h_ref_sel = o, o_ref, hT, hT_ref
    res = dict(o_err=rel_max_err(o_sel, o_ref_sel), hT_err=rel_max_err(h_sel, h_ref_sel),
               o_nmse=nmse(o_sel, o_ref_sel), hT_nmse=nmse(h_sel, h_ref_sel))
    assert res["o_err"] <= tol, res
    assert res["hT_err"] <= tol, res
    return res
