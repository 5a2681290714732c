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
# workload -> number of consecutive steps run (weights carried from step to step; mlp_greedy: batches per
# phase of its layer-by-layer epoch).  Every step of a short run is digested; of a long run the first two
# steps and every tenth (out["digested"] lists them).
CASES = {"tiny_mlp": 10, "mlp_greedy": 58, "mlp_lookahead": 50, "cnn": 3, "roofline": 2, "separable": 2}


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
        # the whole layer-by-layer epoch (Sec. III): `steps` distinct batches per phase, phase l trains layer l on
        # the INT8 forward of the earlier layers as trained by their own phases, weights carried through every
        # step.  out["steps"][l] = digests of layer l at the phase steps listed in out["digested"];
        # out["final_W"][l] = digest of layer l's weights after its phase.
        batches = [synth.make_batch(w, SEED, batch_index=i) for i in range(steps)]
        dig = sorted(set(digested_steps(steps) + [steps - 1]))
        out["digested"] = dig
        out["steps"] = [[] for _ in specs]
        clock = [time.time()]

        def on_step(l, i, states):
            if i in dig:
                out["steps"][l].append(layer_digests(states[l], w.B))
            print(f"{name} phase {l} batch {i}: {time.time() - clock[0]:.1f} s", flush=True)
            clock[0] = time.time()

        Wt = O.greedy_epoch(specs, Ws, batches, w.B, on_step)
        out["final_W"] = [digest(W.astype(np.float32)) for W in Wt]
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
