"""Writes tests/golden/oracle_small_case.json from the CPU oracle alone (no CUDA code is imported)."""
import hashlib
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import Oracle, derive_params  # noqa: E402

SHAPE = dict(d=257, r=5, c=16, k=6, W=3, seed=0x5EED)
NCAND, RHO, STEPS = 12, 0.5, 3


def gradients(step: int) -> np.ndarray:
    """Integer-valued gradients from a fixed recipe (every operation of the step is then exact)."""
    W, d = SHAPE["W"], SHAPE["d"]
    w = np.arange(W, dtype=np.int64)[:, None]
    i = np.arange(d, dtype=np.int64)[None, :]
    g = ((i * 37 + w * 101 + step * 53) % 23) - 11
    g[:, (step * 7 + 3) % d] += 400 * (1 if step % 2 == 0 else -1)      # one dominant coordinate per step
    g[:, 100] += 90
    return g.astype(np.float32)


def compute() -> dict:
    o = Oracle(**SHAPE)
    u = np.zeros((SHAPE["W"], SHAPE["d"]), np.float32)
    v = np.zeros_like(u)
    steps = []
    for t in range(STEPS):
        out = o.step(gradients(t), RHO, u, v, NCAND, full=True)
        steps.append(dict(
            out_idx=sorted(int(x) for x in out["out_idx"]),
            out_val=[float(x) for x in out["out_val"][np.argsort(out["out_idx"])]],
            cand=sorted(int(x) for x in out["cand"]),
            table_sha256=hashlib.sha256(np.ascontiguousarray(out["T"]).tobytes()).hexdigest(),
        ))
    return dict(
        shape=SHAPE, ncand=NCAND, rho=RHO,
        hash_params=[[int(x) for x in row] for row in derive_params(SHAPE["seed"], SHAPE["r"])],
        steps=steps,
        state_sha256=hashlib.sha256(u.tobytes() + v.tobytes()).hexdigest(),
    )


if __name__ == "__main__":
    path = os.path.join(HERE, "oracle_small_case.json")
    with open(path, "w") as f:
        json.dump(compute(), f, indent=1)
    print("wrote", path)
