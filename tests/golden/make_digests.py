"""Writes tests/golden/oracle_digests.txt: SHA-256 digests of oracle outputs on fixed seeded inputs.

Run from the repository root:  python tests/golden/make_digests.py
Only the oracle (oracle/) and the seeded input generators are called; nothing here touches the CUDA
library.  The digests freeze the oracle's arithmetic: a change to the generator, the transform, the
rounding or the mixing of Eq. (perturbation) shows up as a changed line, and the commit that changes
it has to say which passage of the paper, or which reading of it, justifies the change.
"""
import hashlib
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2601_12917_b200 import synth  # noqa: E402


def _h(a: np.ndarray) -> str:
    return hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()


def digests():
    out = []
    # raw generator blocks: Philox4x32-10 keyed by (seed, tensor, tag), incl. block indices beyond 2^32
    out.append(("blocks seed=1 tensor=3 tag=1 first=12345 n=4096", _h(oracle.blocks(1, 3, 1, 12345, 4096))))
    out.append(("blocks seed=2^64-1 tensor=7 tag=0 first=2^40+5 n=4096", _h(oracle.blocks(2**64 - 1, 7, 0, 2**40 + 5, 4096))))
    # normals of both word-to-normal mappings
    for bits in (32, 16):
        out.append((f"normals bits={bits} seed=5 tensor=2 tag=0 e0=0 n=8192", _h(oracle.normals(5, 2, 0, bits, 0, 8192))))
    # one full step of a small mixed model in every storage type (perturb +eps, -2 eps, restore+update)
    shapes, ranks = ((24, 16), (1, 12), (16, 24)), (4, 0, 2)
    for name, dt in (("f32", oracle.F32), ("f16", oracle.F16), ("bf16", oracle.BF16), ("f64", oracle.F64)):
        for bits in (32, 16):
            tensors = []
            for l, ((m, n), r) in enumerate(zip(shapes, ranks)):
                U = synth.subspace(m, r, l) if r else None
                w = synth.weights_host(synth.TensorSpec(f"t{l}", m, n, r), l).ravel()
                tensors.append(oracle.OracleTensor(theta=oracle.encode(w, dt), rows=m, cols=n, dtype=dt, U=U))
            o = oracle.OracleZGR(tensors, alpha=0.5, eps=1e-3, scale_mode=oracle.SCALE_UNIT, bits=bits)
            o.perturb(7, 1e-3)
            o.perturb(7, -2e-3)
            o.restore_update(7, 2.31, 2.29, 1e-2)
            out.append((f"step {name} bits={bits}", _h(np.concatenate([np.asarray(t.theta).view(np.uint8).ravel() for t in tensors]))))
            o.sweep_multi([8, 9], [1e-3, -5e-4])
            out.append((f"sweep_multi {name} bits={bits}", _h(np.concatenate([np.asarray(t.theta).view(np.uint8).ravel() for t in tensors]))))
    # compressed coefficients: int8 symmetric and the INT4 form of Sec. 3.4
    G = oracle.coeffs(3, 0, 32, 4, 64)
    q8, s8, z8 = oracle.dtc_quantise(G, 8, True)
    q4, s4, z4 = oracle.dtc_quantise_int4(G)
    out.append(("dtc int8 codes+scales", _h(np.concatenate([q8.view(np.uint8).ravel(), s8.view(np.uint8).ravel()]))))
    out.append(("dtc int4 packed+scales+zeros", _h(np.concatenate([oracle.dtc_pack4(q4).ravel(), s4.view(np.uint8).ravel(), z4.view(np.uint8).ravel()]))))
    return out


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_digests.txt")
    with open(path, "w") as f:
        f.write("# written by tests/golden/make_digests.py from the oracle alone; see that file\n")
        for what, h in digests():
            f.write(f"{h}  {what}\n")
    print("wrote", path)
