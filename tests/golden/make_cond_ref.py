"""Writes tests/golden/cond_ref.json: the condition numbers (oracle.gradient_condition) of the gradient tensors of the
benchmark network, 400-480-3203 with softmax + cross-entropy and with the paper's tanh + squared-error head (Eqs. 1-3),
on the first 8192 patterns of the benchmark batch (seed 2).  The estimates of the weight gradients, which set the
maximum, do not depend on the number of patterns (512, 2048 and 8192 patterns agree to 7 %); the top bias gradient's
grows with it (the label counts in it are exact), and stays below the weight gradients' at the benchmark batch.  Calls only `oracle/` and
the seeded input generators.  Takes a few minutes on 8 cores.

    python tests/golden/make_cond_ref.py
"""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle                     # noqa: E402
import synth_inputs as si         # noqa: E402


def main():
    sizes, n, seed = [400, 480, 3203], 8192, 2
    Ws, bs = si.mlp_params(seed, sizes)
    X, y = si.mlp_batch(seed, sizes, n)
    T = si.mlp_targets(seed, sizes, n)
    cW, cb = oracle.gradient_condition(Ws, bs, X, labels=y)
    sW, sb = oracle.gradient_condition(Ws, bs, X, T=T)
    out = {
        "what": "oracle.gradient_condition of the 400-480-3203 network, seed 2, first 8192 patterns, eps 2^-14, seeds (12345, 12346)",
        "softmax": {"dW": cW, "db": cb}, "sse": {"dW": sW, "db": sb},
        "cond_ref": max(cW + cb + sW + sb),
    }
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "cond_ref.json"), "w") as f:
        json.dump(out, f, indent=1)
        f.write("\n")
    print(json.dumps(out))


if __name__ == "__main__":
    main()
