"""Prints the phase time stamps of the tensor-core kernels from the instrumented build.

    python -m paper_2609_32114_b200.build --profile
    python -m paper_2609_32114_b200.prof_phases [WORKLOAD]          (needs a GPU)

The instrumented library (libha_la_prof.so, -DHA_LA_PROFILE_PHASES) records, for CTA 0 of each kernel, clock64 at
the phase boundaries of its first work items / chunks and a few %globaltimer stamps (kernel start and end, first
and last chunk, when chunks were published).  This script runs one workload through it and prints
  * the chain kernel: cycles per chunk, split into waiting for the operands, the first product, the first
    epilogue, the second product, the second epilogue;
  * the prep kernel: cycles between the numbered phase probes of its first items;
  * a nanosecond timeline of both kernels within one call.
"""
import ctypes
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main(argv):
    import torch

    from paper_2609_32114_b200 import binding, build, synth
    import paper_2609_32114_b200 as ha
    from tests import helpers

    if not os.path.exists(build.PROF_LIB):
        raise SystemExit("build the instrumented library first: python -m paper_2609_32114_b200.build --profile")
    binding.LIB_PATH = build.PROF_LIB
    lib = ha.load_library()
    w = synth.WORKLOADS[argv[1] if len(argv) > 1 else "gdn_layer_4k"]
    inp = synth.make_inputs(w)
    d = helpers.to_device(inp)
    a, keep = ha.prepare_args(d["q"], d["k"], d["v"], d["g"], d["beta"], variant=w.variant, h0=d["h0"],
                              cu_seqlens=d["cu_seqlens"], max_seqlen=d["max_seqlen"])
    s = torch.cuda.current_stream().cuda_stream
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for _ in range(3):
        ha.ha_la_prefill_raw(a, s)
    flush.zero_()
    ha.ha_la_prefill_raw(a, s)
    torch.cuda.synchronize()

    def read(name):
        buf = (ctypes.c_longlong * 1024)()
        getattr(lib, f"ha_la_debug_read_prof_{name}")(buf)
        return np.array(buf[:], dtype=np.int64)

    P, C = read("prep"), read("chain")
    nch = min(64, (max(inp["seq_lens"]) + 63) // 64)
    print("chain kernel, CTA 0, cycles per chunk: operands / product 1 / epilogue 1 / product 2 / epilogue 2 / total")
    for c in list(range(1, min(nch, 9))) + ([nch // 2] if nch > 16 else []):
        t = C[8 * c: 8 * c + 6]
        print(f"  chunk {c:3d}: {t[1]-t[0]:5d} {t[2]-t[1]:5d} {t[3]-t[2]:5d} {t[4]-t[3]:5d} {t[5]-t[4]:5d} {t[5]-t[0]:6d}")
    print("prep kernel, CTA 0 group 0, cycles between phase probes 2..13 of its first items")
    for n in range(3):
        t = P[16 + 16 * n + 2: 16 + 16 * n + 14]
        if t[0] > 0:
            print(f"  item {n}: {[int(x) for x in np.diff(t)]} sum {int(t[-1] - t[0])}")
    t0 = min(P[900], C[900])
    print("timeline (ns from the first kernel's start): prep start", P[900] - t0, "prep end", P[901] - t0,
          "| chain start", C[900] - t0, "first chunk done", C[700] - t0, "last chunk done", C[700 + nch - 1] - t0,
          "chain end", C[901] - t0)
    print("status word:", int(keep["status_word"].item()))


if __name__ == "__main__":
    main(sys.argv)
