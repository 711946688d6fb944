"""Writes tests/golden/tiny_oracle.txt: a digest of the oracle's result on the `tiny` workload.

Calls nothing but oracle/ and the seeded input generators.  The file guards the oracle against
silent change; it is not a value from the paper (the paper prints none).
Run: python tests/golden/make_golden.py
"""
import hashlib
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import numpy as np

import oracle
from paper_2604_26881_b200 import workloads as W


def digest():
    wl = W.WORKLOADS["tiny"]
    wts = W.weights_as_numpy(W.make_weights(wl, seed=0))
    x, tenant, mot = W.make_tokens(wl, seed=0)
    r = oracle.layer_forward(W.as_u16(x), tenant.numpy(), mot.numpy(), wts, k=wl.k, G=wl.G)
    lines = [
        "workload tiny seed 0 (T=64 H=256 E=8 I=128 k=2, no shared expert, G=1)",
        "topk_idx sha256 " + hashlib.sha256(r.routing.topk_idx.tobytes()).hexdigest(),
        "perm sha256 " + hashlib.sha256(r.dispatch.perm.tobytes()).hexdigest(),
        "expert_off " + " ".join(str(int(v)) for v in r.dispatch.expert_off),
        "n_invocations %d" % r.dispatch.n_invocations,
        "flagged_tokens %d" % int(r.routing.tie_flag.sum()),
        "topk_w sum %.12e" % float(r.routing.topk_w.sum()),
        "out sum %.12e" % float(r.out.sum()),
        "out abs sum %.12e" % float(np.abs(r.out).sum()),
        "out[0,:4] " + " ".join("%.12e" % v for v in r.out[0, :4]),
        "out[63,252:] " + " ".join("%.12e" % v for v in r.out[63, 252:]),
    ]
    return "\n".join(lines) + "\n"


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_oracle.txt")
    with open(path, "w") as f:
        f.write(digest())
    print(open(path).read())
