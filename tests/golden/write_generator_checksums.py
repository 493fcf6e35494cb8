"""Writes tests/golden/generator_checksums.json from the seeded input generators.

Calls only the input module (no oracle, no CUDA code).  Run from the repository root:
    python tests/golden/write_generator_checksums.py
"""
import hashlib
import json
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
from paper_2601_12347_b200 import inputs as I  # noqa: E402


def digest(*arrays) -> str:
    h = hashlib.sha256()
    for a in arrays:
        h.update(np.ascontiguousarray(a).tobytes())
    return h.hexdigest()[:32]


SMALL = ("tiny", "sparse", "mid-2l")          # regenerated and compared by the CPU tests
LARGE = ("dense-2l", "reddit-2l")            # compared where the graphs are generated anyway: the full-size GPU tests


def graph_digest(src, dst) -> str:
    return digest(src, dst)


def checksums(names=SMALL):
    out = {}
    for name in names:
        w = I.workloads()[name]
        src, dst = I.make_graph(w)
        X = I.features(w.n, w.model.dims[0], w.seed)
        W = I.make_weights(w.model, w.seed)
        st = I.UpdateStream(w.n, src, dst, w.model.dims[0], w.seed)
        ups, rows = st.next_batch(100)
        deg = np.bincount(src, minlength=w.n)
        out[name] = {
            "edges": int(src.size),
            "graph": graph_digest(src, dst),
            "max_out_degree": int(deg.max()),
            "zero_out_degree": int((deg == 0).sum()),
            "features": digest(X[:64]),
            "weights": digest(*[W[i][k] for i in range(len(W)) for k in sorted(W[i])]),
            "first_batch": digest(ups, rows),
        }
    return out


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "generator_checksums.json")
    with open(path, "w") as f:
        json.dump(checksums(SMALL + LARGE), f, indent=1, sort_keys=True)
    print("wrote", path)
