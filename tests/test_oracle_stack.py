"""Pins for the oracle's stack of coupling branches: what reversibility and the
chain rule fix, checked without reusing the stack code itself."""
import numpy as np

from oracle import revffn_oracle as orc
from workloads import BlockConfig, make_streams, make_weights

TINY = BlockConfig("tiny", tokens=6, d_model=16, n_experts=5, top_k=2, d_expert=12, d_shared=10, weight_dtype="f32")


def _blocks(n, seed=0, scale=10.0):
    out = []
    for l in range(n):
        p = make_weights(TINY, seed, block=l)
        for name in p:
            p[name] = p[name].astype(np.float64)      # fp64 storage, so that a 1e-6 step is not rounded away
            if name != "norm_gamma":
                p[name] = p[name] * scale
        out.append(p)
    return out


def test_stack_is_the_hand_written_composition():
    """Two layers written out by hand: B1 = B0 + F0(A0); A1 = A0 + F1(B1)."""
    blocks, s = _blocks(2), make_streams(TINY, 3)
    A0, B0 = s["y1"].astype(np.float64), s["x2"].astype(np.float64)
    B1, _ = orc.forward(blocks[0], A0, B0, TINY.top_k)
    A1, _ = orc.forward(blocks[1], B1, A0, TINY.top_k)
    A, B, infos = orc.stack_forward(blocks, A0, B0, TINY.top_k)
    assert np.array_equal(A, A1) and np.array_equal(B, B1)
    assert len(infos) == 2
    # a single layer is Eq. 2 itself
    A, B, _ = orc.stack_forward(blocks[:1], A0, B0, TINY.top_k)
    assert np.array_equal(A, A0) and np.array_equal(B, B1)


def test_stack_inverts_exactly_in_fp64():
    blocks, s = _blocks(7), make_streams(TINY, 1)
    A, B, _ = orc.stack_forward(blocks, s["y1"], s["x2"], TINY.top_k)
    assert np.abs(A - s["y1"]).max() > 1e-3 and np.abs(B - s["x2"]).max() > 1e-3   # both streams really change
    A0, B0 = orc.stack_inverse(blocks, A, B, TINY.top_k)
    assert np.max(np.abs(A0 - s["y1"])) <= 1e-10
    assert np.max(np.abs(B0 - s["x2"])) <= 1e-10


def _loss(blocks, A, B, cA, cB):
    A1, B1, infos = orc.stack_forward(blocks, A, B, TINY.top_k)
    return float(np.sum(cA * A1) + np.sum(cB * B1)), infos


def test_stack_backward_matches_central_differences():
    """dLoss/dInputs and one weight per layer against central differences of the
    forward stack (entries whose routing margin is far above the step)."""
    blocks, s = _blocks(3, seed=2), make_streams(TINY, 2)
    rng = np.random.default_rng(0)
    cA, cB = rng.standard_normal(s["y1"].shape), rng.standard_normal(s["x2"].shape)
    A0, B0 = s["y1"].astype(np.float64), s["x2"].astype(np.float64)
    A1, B1, infos = orc.stack_forward(blocks, A0, B0, TINY.top_k)
    assert min(float(i["margin"].min()) for i in infos) > 1e-3
    Ar, Br, dA, dB, grads = orc.stack_backward(blocks, A1, B1, cA, cB, TINY.top_k)
    assert np.max(np.abs(Ar - A0)) <= 1e-10 and np.max(np.abs(Br - B0)) <= 1e-10
    eps = 1e-6
    for _ in range(6):
        t, i = rng.integers(TINY.tokens), rng.integers(TINY.h)
        for X, dX, which in ((A0, dA, "A"), (B0, dB, "B")):
            Xp, Xm = X.copy(), X.copy()
            Xp[t, i] += eps; Xm[t, i] -= eps
            lp, _ = _loss(blocks, Xp if which == "A" else A0, Xp if which == "B" else B0, cA, cB)
            lm, _ = _loss(blocks, Xm if which == "A" else A0, Xm if which == "B" else B0, cA, cB)
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - dX[t, i]) <= 1e-6 * max(1.0, abs(fd)), (which, t, i, fd, dX[t, i])
    for l, name in ((0, "w_up"), (1, "w_downx"), (2, "ws_gate"), (1, "norm_gamma"), (0, "w_router")):
        W = blocks[l][name]
        pos = tuple(int(rng.integers(n)) for n in W.shape)
        old = W[pos]
        W[pos] = old + eps; lp, _ = _loss(blocks, A0, B0, cA, cB)
        W[pos] = old - eps; lm, _ = _loss(blocks, A0, B0, cA, cB)
        W[pos] = old
        fd = (lp - lm) / (2 * eps)
        got = grads[l][name][pos]
        assert abs(fd - got) <= 2e-6 * max(1.0, abs(fd)), (l, name, fd, got)
