#!/usr/bin/env python
"""Writes tests/golden/fullsize_digests.json: SHA-256 digests of every tensor the CPU oracle produces
for train steps at the FULL sizes of the five benchmark configurations (the sizes bench.py times) and of
the separable-convolution block.

Calls only oracle/ and the seeded input generators; nothing here comes from the CUDA path.  The GPU
test tests/test_gpu_fullsize.py recomputes the same digests from the device buffers, so a full-size
step is compared bit for bit without shipping gigabytes of expected values.

    python tests/golden/make_fullsize_digests.py [workload ...]      (minutes of CPU time, ~12 GB RAM)
"""
import hashlib
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import ffint8_oracle as O          # noqa: E402
from paper_2506_22771_b200 import synth        # noqa: E402

OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "fullsize_digests.json")
SEED = 1
# workload -> number of consecutive steps run (weights carried from step to step).  Every step of a short
# run is digested; of a long run the first two steps and every tenth (out["digested"] lists them).
CASES = {"tiny_mlp": 10, "mlp_greedy": 3, "mlp_lookahead": 50, "cnn": 3, "roofline": 2, "separable": 2}


def digested_steps(steps: int):
    return [s for s in range(steps) if steps <= 10 or s < 2 or s % 10 == 9]


def digest(a) -> str:
    return hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()


def layer_digests(st: O.LayerState, B: int) -> dict:
    return {
        "absmax": [float(np.float32(v)).hex() for v in (st.a_x[0], st.a_x[1], st.a_w, st.a_dh[0], st.a_dh[1])],
        "Xq": digest(st.Xq), "Wq": digest(st.Wq), "Y": digest(st.Y.astype(np.float32)),
        "S": digest(st.S.astype(np.uint64)), "rowmax": digest(st.rowmax.astype(np.int32)),
        "G": digest(st.G.astype(np.float32)), "coef": digest(st.coef.astype(np.float32)),
        "dHq": digest(st.dHq), "W_new": digest(st.W_new.astype(np.float32)), "loss": float(st.loss),
    }


def run(name: str, steps: int) -> dict:
    w = synth.workload(name)
    specs = [O.LayerSpec(l.kind, l.K, l.N, l.theta, l.lr, l.tau, l.eps, l.H, l.Wd, l.Cin, seed=SEED, index=i,
                         stride=l.stride, momentum=l.momentum) for i, l in enumerate(w.layers)]
    Ws = synth.make_weights(w, SEED)
    X = synth.make_batch(w, SEED)
    out = {"B": w.B, "seed": SEED, "greedy": bool(w.greedy), "n_steps": steps, "digested": digested_steps(steps),
           "steps": []}
    if w.greedy:
        # layers trained one after another (Sec. III): phase l trains layer l alone on the INT8 forward of
        # the earlier layers; here every phase starts from the initial weights so that it can be checked on
        # its own.  out["steps"][l][step] = digests of layer l.
        for l, spec in enumerate(specs):
            Wl = Ws[l]
            phase = []
            for step in range(steps):
                t0 = time.time()
                x = X
                for j in range(l):
                    x = O.layer_forward(specs[j], x, Ws[j], w.B, step).Xnext
                st = O.train_step([spec], [Wl], x, w.B, 0.0, step)[0]
                phase.append(layer_digests(st, w.B))
                Wl = st.W_new
                print(f"{name} layer {l} step {step}: {time.time() - t0:.1f} s", flush=True)
            out["steps"].append(phase)
        return out
    for step in range(steps):
        t0 = time.time()
        states = O.train_step(specs, Ws, X, w.B, w.lam_per_step * step, step)
        if step in out["digested"]:
            out["steps"].append([layer_digests(st, w.B) for st in states])
        Ws = [st.W_new for st in states]
        print(f"{name} step {step}: {time.time() - t0:.1f} s", flush=True)
    return out


if __name__ == "__main__":
    names = sys.argv[1:] or list(CASES)
    data = json.load(open(OUT)) if os.path.exists(OUT) else {}
    for n in names:
        data[n] = run(n, CASES[n])
        json.dump(data, open(OUT, "w"), indent=1, sort_keys=True)
    print("wrote", OUT)
