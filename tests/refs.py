"""Second, deliberately different evaluators used only to pin the CPU checker: double
precision, index arithmetic written another way (padded copies instead of skipped taps,
channel-first loops), no code shared with oracle/."""
import numpy as np


def conv_brute(x, w, bias, stride, pad, groups, res=None, act="none"):
    """float64 result before the fp16 rounding.  x NHWC, w [co][kh][kw][cg]."""
    x = x.astype(np.float64)
    w = w.astype(np.float64)
    n, h, wd, cin = x.shape
    cout, kh, kw, cg = w.shape
    xp = np.zeros((n, h + 2 * pad, wd + 2 * pad, cin))
    xp[:, pad:pad + h, pad:pad + wd, :] = x
    ho = (h + 2 * pad - kh) // stride + 1
    wo = (wd + 2 * pad - kw) // stride + 1
    og = cout // groups
    y = np.zeros((n, ho, wo, cout))
    for b in range(n):
        for co in range(cout):
            g = co // og
            for ci in range(cg):
                for i in range(ho):
                    for j in range(wo):
                        for s in range(kw):
                            for r in range(kh):
                                y[b, i, j, co] += (xp[b, i * stride + r, j * stride + s, g * cg + ci]
                                                   * w[co, r, s, ci])
    y += bias.astype(np.float64)[None, None, None, :]
    if res is not None:
        y += res.astype(np.float64)
    return activate(y, act)


def activate(y, act):
    if act == "relu":
        return np.maximum(y, 0.0)
    if act == "relu6":
        return np.minimum(np.maximum(y, 0.0), 6.0)
    return y


def pool2(y):
    n, h, w, c = y.shape
    y = y[:, :h // 2 * 2, :w // 2 * 2, :]
    return y.reshape(n, h // 2, 2, w // 2, 2, c).max(axis=(2, 4))


def ulp_diff(a16, b16):
    """Distance in fp16 steps between two finite fp16 arrays (sign-magnitude ordered)."""
    def key(v):
        u = v.view(np.uint16).astype(np.int32)
        return np.where(u & 0x8000, -(u & 0x7FFF), u & 0x7FFF)
    return np.abs(key(np.ascontiguousarray(a16)) - key(np.ascontiguousarray(b16)))


def assert_matches_exact_math(got16, ref64, min_exact=0.97):
    """got16 came from fp32 accumulation + one rounding; ref64 is the exact value.  They may
    differ by one fp16 step where the exact value sits next to a rounding boundary."""
    want = ref64.astype(np.float16)
    d = ulp_diff(got16, want)
    assert d.max() <= 1, d.max()
    assert (d == 0).mean() >= min_exact, (d == 0).mean()
