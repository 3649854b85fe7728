import os


def load_paper_values():
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "paper_values.txt")
    out = {}
    with open(path) as fh:
        for line in fh:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            key, val = (s.strip() for s in line.split("=", 1))
            out[key] = float(val)
    return out


ABS_TOL = 2e-2   # max abs error against fp64 (spec tolerance)
REL_TOL = 1e-2   # max rel error against fp64


def assert_close_to_oracle(got, ref, what=""):
    """bf16-in / fp32-accumulate outputs against the fp64 oracle: max abs error <= 2e-2 and
    max rel error <= 1e-2.  The relative error of an element whose reference is (nearly)
    zero is taken against max(|ref|, 1e-3 * rms(ref)); how many elements needed that floor
    is returned so callers can report it."""
    import numpy as np
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - ref)
    rms = float(np.sqrt((ref * ref).mean())) if ref.size else 0.0
    floor = 1e-3 * rms
    denom = np.maximum(np.abs(ref), floor)
    denom[denom == 0] = 1.0
    rel = err / denom
    assert err.max(initial=0.0) <= ABS_TOL, f"{what}: max abs err {err.max():.3e}"
    assert rel.max(initial=0.0) <= REL_TOL, f"{what}: max rel err {rel.max():.3e}"
    return int((np.abs(ref) < floor).sum())


def assert_chain_close(got, ref, what=""):
    """Outputs of a CHAIN of kernels with bf16 tensors in between (a whole decode step).
    One bf16 rounding that falls the other way on the two sides moves an intermediate by
    2^-8 relative and every output by about that fraction of the output's typical size, so
    element-wise relative error near zero crossings is not meaningful here: the error is
    bounded by 2e-2 absolute and by 1e-2 of max(|ref|, rms(ref)).  Each kernel of the chain
    is held to the strict tolerance in its own test."""
    import numpy as np
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape and np.isfinite(got).all(), what
    err = np.abs(got - ref)
    rms = float(np.sqrt((ref * ref).mean())) if ref.size else 0.0
    denom = np.maximum(np.abs(ref), rms if rms > 0 else 1.0)
    assert err.max(initial=0.0) <= ABS_TOL, f"{what}: max abs err {err.max():.3e}"
    assert (err / denom).max(initial=0.0) <= REL_TOL, f"{what}: max err / max(|ref|, rms) {(err / denom).max():.3e}"
