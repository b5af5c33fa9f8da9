"""Arithmetic pins of the vision-encoding stage oracle (Sec. 3.3, Eq. 5-7): values worked out by
hand, not by the functions under test.

The paper fixes neither the similarity measure, the weights, tau nor the fence, so the *reading*
cannot be pinned to it; what is pinned here is the arithmetic of the reading taken: mean (not sum)
of the six pair cosines of a 2 x 2 window, strict "> tau", plain (not norm-weighted) average placed
at the window's first raster slot, linearly interpolated quartiles, fence factor 1.5, strict "> mu".
The last test plants each of those mistakes in a copy of the oracle's source and checks that the
pins above catch it.
"""
import math
import os
import types

import numpy as np
import pytest

from oracle import context

E = np.eye(4)


def _grid_4x4():
    """A 4 x 4 grid (4 channels) whose four 2 x 2 windows have cosines known exactly.

    window 0 (slots 0, 1, 4, 5):    four copies of one vector           -> six cosines of 1, S = 1
    window 1 (slots 2, 3, 6, 7):    (2,0,0,0) (1,0,0,0) (1,0,0,0) (0,1,0,0)
                                     -> three cosines of 1, three of 0: S = 3/6 = 0.5 exactly
    window 2 (slots 8, 9, 12, 13):  the four unit vectors              -> S = 0
    window 3 (slots 10, 11, 14, 15): e0, -e0, e1, -e1                   -> cosines -1, 0, 0, 0, 0, -1: S = -1/3
    """
    x = np.zeros((16, 4))
    x[[0, 1, 4, 5]] = [3.0, -1.0, 0.5, 2.0]
    x[2], x[3], x[6], x[7] = 2 * E[0], E[0], E[0], E[1]
    x[8], x[9], x[12], x[13] = E[0], E[1], E[2], E[3]
    x[10], x[11], x[14], x[15] = E[0], -E[0], E[1], -E[1]
    return x


def pin_lsm_similarities(ctx):
    _, _, sims = ctx.local_spatial_merge(_grid_4x4(), 4, 2, tau=0.8, return_sims=True)
    assert sims.shape == (4,)
    assert abs(sims[0] - 1.0) < 1e-15
    assert sims[1] == 0.5                      # the MEAN of three ones and three zeros (their sum is 3)
    assert sims[2] == 0.0
    assert abs(sims[3] + 1.0 / 3.0) < 1e-15    # signed cosines (absolute values would give +1/3)


def pin_lsm_threshold_is_strict(ctx):
    x = _grid_4x4()
    m, slots = ctx.local_spatial_merge(x, 4, 2, tau=0.5)            # S = 0.5 is not > 0.5
    assert m.shape[0] == 13 and list(slots) == [0] + list(range(2, 4)) + list(range(6, 16))
    m, slots = ctx.local_spatial_merge(x, 4, 2, tau=0.49)           # 0.5 > 0.49: window 1 merges too
    assert m.shape[0] == 10 and list(slots) == [0, 2] + list(range(8, 16))
    # between the mean (0.5) and the sum (3) of the pair cosines only the mean decides
    m, _ = ctx.local_spatial_merge(x, 4, 2, tau=0.6)
    assert m.shape[0] == 13


def pin_lsm_merged_token(ctx):
    x = _grid_4x4()
    m, slots = ctx.local_spatial_merge(x, 4, 2, tau=0.49)
    # window 0 -> its common vector at slot 0; window 1 -> the PLAIN average at its first slot, 2:
    # ((2 + 1 + 1 + 0) / 4, (0 + 0 + 0 + 1) / 4) = (1.0, 0.25); weights by norm would give (1.2, 0.2)
    assert slots[0] == 0 and np.array_equal(m[0], [3.0, -1.0, 0.5, 2.0])
    assert slots[1] == 2 and np.array_equal(m[1], [1.0, 0.25, 0.0, 0.0])
    # the untouched windows keep their tokens, bit for bit, in raster order
    assert np.array_equal(m[2:], x[8:16])
    # nothing merges at a tau no similarity exceeds; everything with S > tau merges at tau < -1/3
    assert ctx.local_spatial_merge(x, 4, 2, tau=1.0)[0].shape[0] == 16
    m_all, s_all = ctx.local_spatial_merge(x, 4, 2, tau=-0.5)
    assert list(s_all) == [0, 2, 8, 10] and np.array_equal(m_all[2], [0.25, 0.25, 0.25, 0.25])
    assert np.array_equal(m_all[3], [0.0, 0.0, 0.0, 0.0])


def pin_fence_on_elements(ctx):
    # nine values: the quartiles sit at positions (9 - 1) / 4 = 2 and 6 of the sorted list
    a = np.array([3.0, 16.0, 0.0, 5.0, 12.0, 1.0, 6.0, 2.0, 4.0])   # sorted: 0 1 2 3 4 5 6 12 16
    # Q1 = 2, Q3 = 6, mu = 6 + 1.5 * 4 = 12
    assert ctx.upper_fence(a) == 12.0


def pin_fence_interpolates(ctx):
    # eight values: positions 7 / 4 = 1.75 and 5.25 -> Q1 = 1.75, Q3 = 5.25 on 0..6 and one large value
    a = np.array([4.0, 0.0, 6.0, 2.0, 40.0, 1.0, 5.0, 3.0])
    # mu = 5.25 + 1.5 * 3.5 = 10.5   (nearest-rank quartiles 2 and 5 would give 9.5)
    assert ctx.upper_fence(a) == 10.5


def _rank_one_case(M, t):
    """Keys whose logits are written down directly: D = 4, q_cls[h] = (2, 0, 0, 0), so the logit
    of token j under head h is 2 * k[h][j][0] / sqrt(4) = k[h][j][0] = t[h][j]."""
    H = len(t)
    q = np.zeros((H, 4))
    q[:, 0] = 2.0
    k = np.zeros((H, M, 4))
    for h in range(H):
        k[h, :, 0] = t[h]
        k[h, :, 1:] = 7.0 * (h + 1)            # orthogonal to q_cls: must not matter
    a = []
    for j in range(M):
        acc = 0.0
        for h in range(H):
            acc += math.exp(t[h][j]) / sum(math.exp(x) for x in t[h])
        a.append(acc / H)
    return q, k, a


def _fence_by_hand(a):
    s = sorted(a)
    n = len(s)

    def quartile(p):
        pos = (n - 1) * p
        lo = int(math.floor(pos))
        hi = min(lo + 1, n - 1)
        return s[lo] + (pos - lo) * (s[hi] - s[lo])

    q1, q3 = quartile(0.25), quartile(0.75)
    return q3 + 1.5 * (q3 - q1), q1, q3


def pin_key_set_rank_one(ctx):
    # M = 9 (quartiles on elements) and M = 8 (interpolated); two heads with different logits
    for M in (9, 8):
        t = [[0.1 * j for j in range(M)], [0.05 * (M - j) for j in range(M)]]
        t[0][4] += 3.0                          # one token far above the rest under both heads
        t[1][4] += 2.5
        q, k, a = _rank_one_case(M, t)
        O, a_got = ctx.key_set(q, k)
        assert np.allclose(a_got, a, rtol=1e-13, atol=0)
        assert abs(sum(a) - 1.0) < 1e-14
        mu, q1, q3 = _fence_by_hand(a)
        assert abs(ctx.upper_fence(np.array(a)) - mu) <= 1e-15
        want = [j for j in range(M) if a[j] > mu]
        assert want == [4] and list(O) == want
        # the fence factor matters in this case: at 3.0 (the "far out" fence) ... still an outlier;
        # at a factor that puts the fence above a[4] it is not - so check the number itself
        assert (a[4] - q3) / (q3 - q1) > 1.5


def pin_key_set_strictness_and_factor(ctx):
    # a token exactly AT the fence stays out; one just above is in.  The values are handed to
    # key_set's threshold step directly (softmax values cannot be placed on the fence exactly).
    a = np.array([0.0, 1.0, 2.0, 3.0, 4.0, 5.0, 6.0, 12.0, 16.0])      # mu = 12 (see above)
    mu = ctx.upper_fence(a)
    assert list(np.nonzero(a > mu)[0]) == [8]
    # 13 lies between the fences at 1.5 IQR (12) and 3 IQR (18): an outlier at 1.5 only
    b = np.array([0.0, 1.0, 2.0, 3.0, 4.0, 5.0, 6.0, 13.0, 7.0])        # sorted: 0..7, 13: Q1 = 2, Q3 = 6
    assert ctx.upper_fence(b) == 12.0 and list(np.nonzero(b > ctx.upper_fence(b))[0]) == [7]
    # the same through key_set: logits log(a_j) give a softmax proportional to a_j
    vals = np.array([1.0, 2.0, 3.0, 4.0, 5.0, 6.0, 7.0, 14.0, 8.0])    # Q1 = 3, Q3 = 7, mu = 13 < 14 < 19
    q, k, a2 = _rank_one_case(9, [[math.log(v) for v in vals]])
    O, _ = ctx.key_set(q, k)
    assert list(O) == [7]
    vals[7] = 12.5                                                     # below the fence at 13
    q, k, _ = _rank_one_case(9, [[math.log(v) for v in vals]])
    assert list(ctx.key_set(q, k)[0]) == []


PINS = [pin_lsm_similarities, pin_lsm_threshold_is_strict, pin_lsm_merged_token, pin_fence_on_elements,
        pin_fence_interpolates, pin_key_set_rank_one, pin_key_set_strictness_and_factor]


@pytest.mark.parametrize("pin", PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin(context)


def pin_key_set_token_at_the_fence(ctx):
    """key_set's own comparison is strict: replace its threshold by a value of a_cls itself."""
    vals = np.array([1.0, 2.0, 3.0, 4.0, 5.0, 6.0, 7.0, 14.0, 8.0])
    q, k, a = _rank_one_case(9, [[math.log(v) for v in vals]])
    saved = ctx.upper_fence
    try:
        ctx.upper_fence = lambda arr: float(np.asarray(arr)[7])        # the fence sits exactly on token 7
        assert list(ctx.key_set(q, k)[0]) == []
        ctx.upper_fence = lambda arr: float(np.nextafter(np.asarray(arr)[7], 0.0))
        assert list(ctx.key_set(q, k)[0]) == [7]
    finally:
        ctx.upper_fence = saved


def test_key_set_comparison_is_strict():
    pin_key_set_token_at_the_fence(context)


# ---- planted mistakes: every one of them must fail at least one pin -----------------------------
MISTAKES = {
    "sum of the pair cosines instead of their mean": [("np.mean(sims)", "np.sum(sims)")],
    ">= tau instead of > tau": [("np.mean(sims) > tau", "np.mean(sims) >= tau")],
    "average weighted by the token norms": [
        ("x[ids].mean(axis=0)",
         "np.average(x[ids], axis=0, weights=np.linalg.norm(x[ids], axis=1) + 1e-300)")],
    "merged token at the window's last slot": [("slots.append(ids[0])", "slots.append(ids[-1])")],
    "absolute cosines": [("float(unit[a] @ unit[b])", "abs(float(unit[a] @ unit[b]))")],
    "dot products instead of cosines": [("float(unit[a] @ unit[b])", "float(x[a] @ x[b])")],
    "fence at 3 IQR": [("1.5 * (q3 - q1)", "3.0 * (q3 - q1)")],
    "nearest-rank quartiles": [("[0.25, 0.75])", "[0.25, 0.75], method='nearest')")],
    "fence below the first quartile": [("q3 + 1.5", "q1 + 1.5")],
    ">= mu instead of > mu": [("a > mu", "a >= mu")],
    "head maximum instead of head mean": [("p.mean(axis=0)", "p.max(axis=0)")],
    "no 1/sqrt(d) scale": [("/ np.sqrt(q.shape[-1])", "")],
}


def _mutant(replacements):
    path = os.path.join(os.path.dirname(context.__file__), "context.py")
    with open(path) as f:
        src = f.read()
    for old, new in replacements:
        assert src.count(old) >= 1, "the planted mistake no longer matches the oracle's source: %r" % old
        src = src.replace(old, new)
    mod = types.ModuleType("context_mutant")
    exec(compile(src, path + " (mutant)", "exec"), mod.__dict__)
    return mod


@pytest.mark.parametrize("name", sorted(MISTAKES), ids=lambda n: n.replace(" ", "_"))
def test_planted_mistake_is_caught(name):
    mutant = _mutant(MISTAKES[name])
    caught = []
    for pin in PINS + [pin_key_set_token_at_the_fence]:
        try:
            pin(mutant)
        except AssertionError:
            caught.append(pin.__name__)
    assert caught, "no pin notices: " + name
