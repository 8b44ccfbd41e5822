"""Pins for the whole-block oracle (Sec. 3.1: Eq. 1 followed by Eq. 2, the inverse pass, reversible
back-propagation): central differences through both branches, exact invertibility in fp64, and the
stack against central differences of its own forward pass."""
import numpy as np

from oracle import revffn_block_oracle as blk

H, D, NH, NKV, S, B = 8, 16, 4, 2, 5, 2
E, K, I, IS = 5, 2, 12, 8
CFG = dict(seq_len=S, n_heads=NH, n_kv_heads=NKV, top_k=K, theta=100.0)


def _attn_weights(rng, std):
    dkv = NKV * (D // NH)
    n = lambda *s: rng.standard_normal(s) * std
    return {"norm_gamma": 1.0 + 0.1 * rng.standard_normal(H), "w_up": n(D, H), "w_down": n(H, D), "w_q": n(D, D),
            "b_q": n(D), "w_k": n(dkv, D), "b_k": n(dkv), "w_v": n(dkv, D), "b_v": n(dkv), "w_o": n(D, D)}


def _moe_weights(rng, std):
    n = lambda *s: rng.standard_normal(s) * std
    return {"norm_gamma": 1.0 + 0.1 * rng.standard_normal(H), "w_up": n(D, H), "w_down": n(H, D), "w_router": n(E, D),
            "w_gate": n(E, I, D), "w_upx": n(E, I, D), "w_downx": n(E, D, I), "ws_gate": n(IS, D), "ws_up": n(IS, D),
            "ws_down": n(D, IS), "ws_sgate": n(D)}


def _setup(seed, std=0.3, layers=1):
    rng = np.random.default_rng(seed)
    blocks = [(_attn_weights(rng, std), _moe_weights(rng, std)) for _ in range(layers)]
    T = B * S
    return blocks, rng.standard_normal((T, H)), rng.standard_normal((T, H)), rng.standard_normal((T, H)), \
        rng.standard_normal((T, H))


def test_block_is_exactly_invertible_once_the_fixed_point_has_converged():
    (blocks, X1, X2, _, _) = _setup(0, std=0.12)
    pa, pm = blocks[0]
    Y1, Y2, info = blk.forward(pa, pm, X1, X2, CFG)
    assert not np.allclose(Y1, X1) and not np.allclose(Y2, X2)
    R1, R2 = blk.inverse(pa, pm, Y1, Y2, CFG, n_iter=60)
    assert np.abs(R2 - X2).max() < 1e-10           # Eq. 2 inverts in closed form
    assert np.abs(R1 - X1).max() < 1e-10           # Eq. 1 through the converged iteration
    e1 = np.linalg.norm(blk.inverse(pa, pm, Y1, Y2, CFG, n_iter=1)[0] - X1)
    e0 = np.linalg.norm(Y1 - X1)
    assert 1e-12 < e1 < 0.5 * e0                   # one iteration helps but is not exact


def _loss(blocks, X1, X2, g1, g2, overrides):
    Y1, Y2, _ = blk.stack_forward(blocks, X1, X2, CFG, overrides)
    return float(np.sum(Y1 * g1) + np.sum(Y2 * g2))


def _check_fd(blocks, X1, X2, g1, g2, dX1, dX2, grads, overrides, seed):
    rng = np.random.default_rng(seed)
    eps = 1e-6

    def fd(arr, idx):
        old = arr[idx]
        arr[idx] = old + eps; up = _loss(blocks, X1, X2, g1, g2, overrides)
        arr[idx] = old - eps; dn = _loss(blocks, X1, X2, g1, g2, overrides)
        arr[idx] = old
        return (up - dn) / (2 * eps)

    for grad, arr in ((dX1, X1), (dX2, X2)):
        for _ in range(5):
            idx = tuple(rng.integers(0, s) for s in arr.shape)
            num = fd(arr, idx)
            assert abs(num - grad[idx]) <= 2e-6 * max(1.0, abs(num)), (idx, num, grad[idx])
    for l, (pa, pm) in enumerate(blocks):
        for p, g in ((pa, grads[l][0]), (pm, grads[l][1])):
            for name in p:
                for _ in range(2):
                    idx = tuple(rng.integers(0, s) for s in p[name].shape)
                    num = fd(p[name], idx)
                    assert abs(num - g[name][idx]) <= 2e-6 * max(1.0, abs(num)), (l, name, idx, num, g[name][idx])


def test_block_backward_matches_central_differences_through_both_branches():
    blocks, X1, X2, g1, g2 = _setup(1)
    pa, pm = blocks[0]
    Y1, Y2, info = blk.forward(pa, pm, X1, X2, CFG)
    ov = [info["idx"]]                              # the selection is piecewise constant: hold it while differencing
    _, _, dX1, dX2, ga, gm = blk.backward(pa, pm, Y1, Y2, g1, g2, CFG, route_override=ov[0], exact_inputs=(X1, X2))
    _check_fd(blocks, X1, X2, g1, g2, dX1, dX2, [(ga, gm)], ov, 2)


def test_stack_backward_rebuilds_inputs_and_matches_central_differences():
    blocks, X1, X2, g1, g2 = _setup(3, std=0.1, layers=3)
    Y1, Y2, infos = blk.stack_forward(blocks, X1, X2, CFG)
    ov = [i["idx"] for i in infos]
    R1, R2, dX1, dX2, grads = blk.stack_backward(blocks, Y1, Y2, g1, g2, CFG, n_iter=60, route_overrides=ov)
    assert np.abs(R1 - X1).max() < 1e-10 and np.abs(R2 - X2).max() < 1e-10
    _check_fd(blocks, X1, X2, g1, g2, dX1, dX2, grads, ov, 4)
    # with the paper's single iteration the rebuilt inputs, and with them the gradients, are only approximate
    Q1, _, qX1, _, _ = blk.stack_backward(blocks, Y1, Y2, g1, g2, CFG, n_iter=1, route_overrides=ov)
    assert 1e-12 < np.abs(Q1 - X1).max() < 1e-2
    assert 0 < np.abs(qX1 - dX1).max() < 1e-2 * np.abs(dX1).max()
