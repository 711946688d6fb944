"""The oracle still gives what the committed digest of the `tiny` workload records."""
import importlib.util
import os

HERE = os.path.dirname(os.path.abspath(__file__))


def test_tiny_oracle_digest_unchanged():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    want = open(os.path.join(HERE, "golden", "tiny_oracle.txt")).read().splitlines()
    got = mod.digest().splitlines()
    assert len(got) == len(want)
    for g, w in zip(got, want):
        if " sum " in w or w.startswith("out["):
            # floating-point lines: same to 1e-10 relative (libm differences between hosts)
            wv = [float(v) for v in w.split() if _isnum(v)]
            gv = [float(v) for v in g.split() if _isnum(v)]
            assert len(gv) == len(wv)
            for a, b in zip(gv, wv):
                assert abs(a - b) <= 1e-10 * max(1.0, abs(b)), (g, w)
        else:
            assert g == w


def _isnum(v):
    try:
        float(v)
        return "e" in v or "." in v
    except ValueError:
        return False
