"""Host-side formulas and the tuning heuristic, restated step by step from the paper.

TEST INFRASTRUCTURE ONLY: the product never imports this module.

  * Eq. 1 / Eq. 2: operation counts of a convolution / fully connected layer.
  * Eq. 3: operation intensity = operations / total size of the tensors touched.
  * Eq. 4: size of the joint (fusion scheme, core count) search space.
  * Eq. 5: per-layer core count from channel size and operation count.
  * Algorithm 1: one pass over the layers that closes a fusion block when the operations
    per core reach the critical count, and gives the block 2^floor(log2(average MP)) cores.
  * Sec. V "Oracle Case": exhaustive search over a reduced space of plans.

Algorithm 1's numerical outputs are PARITY UNPINNED: the paper prints no worked example
of a plan.  What is pinned (tests): the operation counts against Table 2 and the layers
quoted in Sec. IV-A/IV-B, Eq. 4 against the printed 8.17e75, and structural limits of the
pass (threshold -> 0 gives one block per parametrised layer, threshold -> infinity one
block per forced segment, monotone block count).

Readings where the printed algorithm is ambiguous (each is stated where it is used):
the running sum of MPs is kept apart from its mean; the mean is not formed while a block
holds no convolution / FC layer; indices run 0..n-1; a block's end index is inclusive and
the tail is always closed; a caller-supplied rule can force a block to close; a block whose
average MP reaches the core count of the chip gets the whole chip (the paper's top step, 32, is
its whole chip; on a chip whose core count is not a power of two the floor would leave cores idle).
"""
from __future__ import annotations

import math
from itertools import product


# ---- Eq. 1, Eq. 2, Eq. 3 --------------------------------------------------------------

def eq1_conv_ops(h_out, w_out, h_k, w_k, c_in, c_out):
    """Eq. 1, literally: 2 * H_out * W_out * H_K * W_K * C_in * C_out (no batch, no groups)."""
    return 2 * h_out * w_out * h_k * w_k * c_in * c_out


def eq2_fc_ops(m, k, n):
    """Eq. 2: 2 * M * K * N."""
    return 2 * m * k * n


def eq3_intensity(ops, tensor_bytes):
    """Eq. 3: operations divided by the summed size of the tensors."""
    return ops / float(sum(tensor_bytes))


def infer_shapes(layers, n, h, w, c):
    """Output shape (n, h, w, c) of every layer; floor division as in the usual definition of
    a strided convolution's output size."""
    shapes = []
    for l in layers:
        sh = (n, h, w, c) if l["src"] < 0 else shapes[l["src"]]
        if l["op"] in ("conv", "dwconv", "maxpool"):
            ho = (sh[1] + 2 * l["pad"] - l["kh"]) // l["stride"] + 1
            wo = (sh[2] + 2 * l["pad"] - l["kw"]) // l["stride"] + 1
            if l.get("pool", 0) == 2:
                ho, wo = ho // 2, wo // 2
            shapes.append((sh[0], ho, wo, l["cout"] if l["op"] != "maxpool" else sh[3]))
        elif l["op"] == "gavgpool":
            shapes.append((sh[0], 1, 1, sh[3]))
        elif l["op"] == "fc":
            shapes.append((sh[0], 1, 1, l["cout"]))
        else:
            raise ValueError(l["op"])
    return shapes


def layer_ops(layers, n, h, w, c, literal=False):
    """Per-layer operation counts (0 for layers without weights).

    literal=True applies Eq. 1 exactly as printed (no batch, depthwise counted as dense;
    Eq. 2 with M = 1 row), which is what reproduces Table 2.  literal=False is the work
    of one launch: times the batch, divided by the groups."""
    shapes = infer_shapes(layers, n, h, w, c)
    out = []
    for l, sh in zip(layers, shapes):
        if l["op"] in ("conv", "dwconv"):
            src = (n, h, w, c) if l["src"] < 0 else shapes[l["src"]]
            ho = (src[1] + 2 * l["pad"] - l["kh"]) // l["stride"] + 1  # before any fused pool
            wo = (src[2] + 2 * l["pad"] - l["kw"]) // l["stride"] + 1
            ops = eq1_conv_ops(ho, wo, l["kh"], l["kw"], l["cin"], l["cout"])
            out.append(ops if literal else ops * sh[0] // l["groups"])
        elif l["op"] == "fc":
            out.append(eq2_fc_ops(1 if literal else sh[0], l["cin"], l["cout"]))
        else:
            out.append(0)
    return out


# ---- Eq. 4 ----------------------------------------------------------------------------

def eq4_space(n, q=32):
    """Eq. 4: sum over i = 1..n-1 cut points of q^(i+1) * C(n-1, i)."""
    return sum(q ** (i + 1) * math.comb(n - 1, i) for i in range(1, n))


def enumerate_plans(n, choices):
    """Every (group_end list, core count list): all contiguous partitions of n layers, each
    block with one of `choices`.  There are q (q+1)^(n-1) of them; Eq. 4 leaves out the q
    single-block ones."""
    for cuts in product((0, 1), repeat=n - 1):
        ends = [i for i in range(n - 1) if cuts[i]] + [n - 1]
        for mps in product(choices, repeat=len(ends)):
            yield ends, list(mps)


# ---- Eq. 5 ----------------------------------------------------------------------------

def eq5_score(c, op_count, alpha, beta):
    """Right-hand side of Eq. 5: alpha * log2(C) + beta * log2(OpCount)."""
    return alpha * math.log2(c) + beta * math.log2(op_count)


def layer_mp(c, op_count, p):
    """Eq. 5 gives a proportionality only; reading: an affine map of the score, rounded to
    the nearest integer (halves away from zero) and clamped to [1, s_max]."""
    s = p["kappa"] * eq5_score(c, op_count, p["alpha"], p["beta"]) + p["kappa0"]
    return int(min(max(math.floor(s + 0.5), 1), p["s_max"]))


# ---- Algorithm 1 ----------------------------------------------------------------------

def algorithm1(kinds, channels, ops, p, must_close_after=None, may_close=None):
    """kinds[i]: True when layer i is a convolution / fully connected layer; channels[i],
    ops[i]: its C and operation count (ignored otherwise).  p: dict with alpha, beta,
    kappa, kappa0, s_max, op_critical.  must_close_after(start, i) -> bool forces the block
    that started at `start` to end at layer i; may_close(start, i) -> bool says whether the layers
    start..i already form a block that can run (a block whose layers are only the beginning of a
    fusable pattern keeps growing past the threshold).  Returns (partition_index, mp_of_block)."""
    n = len(kinds)
    partition, mp_of_block = [], []
    sum_op, sum_mp, block_size, start = 0.0, 0.0, 0, 0
    for i in range(n):
        if kinds[i]:
            current_mp = layer_mp(channels[i], ops[i], p)
            sum_op += ops[i]
            sum_mp += current_mp
            block_size += 1
        forced = (i == n - 1) or (must_close_after is not None and must_close_after(start, i))
        if block_size > 0:
            avg_mp = sum_mp / block_size
            closable = may_close is None or may_close(start, i)
            if (sum_op / avg_mp >= p["op_critical"] and closable) or forced:
                partition.append(i)
                mp = 2 ** int(math.floor(math.log2(avg_mp)))
                if avg_mp >= p["s_max"]:  # the top step is the whole chip (32 of 32 cores in the paper)
                    mp = p["s_max"]
                mp_of_block.append(int(min(max(mp, 1), p["s_max"])))
                sum_op, sum_mp, block_size, start = 0.0, 0.0, 0, i + 1
        elif forced:  # a block of layers without weights (a pool on its own)
            partition.append(i)
            mp_of_block.append(int(p["s_max"]))
            start = i + 1
    return partition, mp_of_block


# ---- reduced brute force (Sec. V, "Oracle Case") -----------------------------------------

def best_plan_exhaustive(n, choices, group_time, max_len=None):
    """Tries every plan of `enumerate_plans` whose blocks are allowed (group_time returns a
    float, or None for a block that cannot run) and returns (best_time, ends, mps).  A
    plan's time is the sum of its blocks' times."""
    best = (math.inf, None, None)
    for ends, mps in enumerate_plans(n, choices):
        t, a, ok = 0.0, 0, True
        for e, m in zip(ends, mps):
            if max_len is not None and e - a + 1 > max_len:
                ok = False
                break
            g = group_time(a, e, m)
            if g is None:
                ok = False
                break
            t += g
            a = e + 1
        if ok and t < best[0]:
            best = (t, ends, mps)
    return best
