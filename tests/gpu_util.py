"""Shared helpers of the GPU parity tests: run a plan through the C ABI, run the CPU checker on
the same seeded tensors, compare at every group boundary."""
import numpy as np

TOL = 1e-2  # per element: |err| <= TOL * (1 + |ref|); network outputs: relative L2 <= TOL


def compare(got, ref, what=""):
    got = got.astype(np.float64)
    ref = ref.astype(np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.isfinite(got).all(), what + ": non-finite values"
    err = np.abs(got - ref)
    bound = TOL * (1.0 + np.abs(ref))
    bad = err > bound
    if bad.any():
        idx = np.argwhere(bad)
        first = tuple(idx[0])
        raise AssertionError("%s: %d of %d elements off (max err %.4g); first at %s got %.5g want %.5g; "
                             "bad index ranges %s..%s" % (what, bad.sum(), bad.size, err.max(), first, got[first],
                                                          ref[first], idx.min(axis=0), idx.max(axis=0)))
    return float(err.max())


def rel_l2(got, ref):
    got = got.astype(np.float64)
    ref = ref.astype(np.float64)
    return float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30))


def check_plan(sess, x_dev, ref_outs, group_end, sm_count, what=""):
    """Installs the plan, runs once, compares every group-ending layer with the checker."""
    ends, _ = sess.set_plan(group_end, sm_count)
    sess.run(x_dev)
    worst = 0.0
    for e in ends:
        worst = max(worst, compare(sess.boundary(e), ref_outs[e], "%s layer %d (%s)" % (what, e, ",".join(sess.kernels()))))
    r = rel_l2(sess.boundary(ends[-1]), ref_outs[ends[-1]])
    assert r <= TOL, (what, r)
    return worst


def all_contiguous_plans(n):
    for mask in range(1 << (n - 1)):
        yield [i for i in range(n - 1) if mask >> i & 1] + [n - 1]
