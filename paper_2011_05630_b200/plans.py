"""Plan helpers on top of the C ABI: default tuner constants for B200 and the strategies the
benchmark compares.  Everything here only marshals arguments; the tuner (Eq. 5 + Algorithm 1)
and the reduced brute-force search run inside the library."""
from __future__ import annotations

from . import binding as B

# Eq. 5 weights are the paper's; the affine map to an SM count and the critical operation count
# per SM are fitted to B200 (the paper fits them to its own accelerator the same way).
TUNER = dict(alpha=0.316, beta=0.659, kappa=12.0, kappa0=-60.0, op_critical=1.0e7)


def tuned_plan(net, n_layers, **over):
    p = dict(TUNER, **over)
    return B.net_autotune(net, n_layers, p["alpha"], p["beta"], p["kappa"], p["kappa0"], p["op_critical"],
                          s_max=0, legalise=1)


def sm_fractions(sms):
    """The paper's reduced core-count set {1,2,4,8,12,16,24,32}/32 scaled to this device."""
    return sorted({max(1, round(sms * f / 32)) for f in (1, 2, 4, 8, 12, 16, 24, 32)})
