"""Unit tests of the two GEMM back ends (tcgen05 and CUDA-core) through the
debug entry point, against a plain torch fp32 evaluation of the same problem.
Covers every operand layout, concatenation, grouping and epilogue the three
passes use, at sizes that span several tiles and a ragged tail."""
import ctypes as C

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

EPI = dict(store=0, swiglu=1, rowscale=2, couple=3, dswiglu=4, wgrad=5)


@pytest.fixture(scope="module")
def rv():
    import paper_2512_20920_b200 as rv
    return rv


def _bf(shape, seed, scale=1.0):
    g = torch.Generator("cuda").manual_seed(seed)
    return (torch.randn(*shape, device="cuda", generator=g) * scale).to(torch.bfloat16)


def _call(rv, use_simt, **kw):
    from paper_2512_20920_b200.binding import DbgGemmArgs
    a = DbgGemmArgs()
    a.resid_sign = 1.0
    keep = []
    for k, v in kw.items():
        if isinstance(v, torch.Tensor):
            keep.append(v)
            v = v.data_ptr()
        setattr(a, k, v)
    a.use_simt = 1 if use_simt else 0
    status = torch.zeros(64, dtype=torch.int32, device="cuda")
    code = rv.lib.revffn_dbg_gemm(C.byref(a), status.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert code == 0, rv.revffn_strerror(code)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    return keep


def _close(a, b, tol=1e-2):
    a = a.float().cpu().numpy().astype(np.float64)
    b = b.float().cpu().numpy().astype(np.float64)
    err = np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30)
    assert err <= tol, err


BACKENDS = [pytest.param(True, id="simt"), pytest.param(False, id="tcgen05")]


@pytest.mark.parametrize("simt", BACKENDS)
@pytest.mark.parametrize("M,N,K", [(300, 256, 192), (128, 128, 64), (77, 384, 1024), (1000, 512, 128)])
def test_store_k_major(rv, simt, M, N, K):
    A, B = _bf((M, K), 1), _bf((N, K), 2)
    Cb = torch.full((M, N), float("nan"), device="cuda", dtype=torch.bfloat16)
    _call(rv, simt, M=M, N=N, K=K, A=A, B0=B, lda=K, ldb=K, C=Cb, ldc=N, epilogue=EPI["store"])
    _close(Cb, A.float() @ B.float().T)
    Cf = torch.full((M, N), float("nan"), device="cuda", dtype=torch.float32)
    _call(rv, simt, M=M, N=N, K=K, A=A, B0=B, lda=K, ldb=K, C=Cf, ldc=N, epilogue=EPI["store"], out_f32=1)
    _close(Cf, A.float() @ B.float().T, 1e-5)


@pytest.mark.parametrize("simt", BACKENDS)
def test_store_b_mn_major(rv, simt):
    M, N, K = 300, 384, 256
    A, B = _bf((M, K), 3), _bf((K, N), 4)            # B stored [K, N]
    Cf = torch.full((M, N), float("nan"), device="cuda", dtype=torch.float32)
    _call(rv, simt, M=M, N=N, K=K, A=A, B0=B, lda=K, ldb=N, b_mn_major=1, C=Cf, ldc=N, epilogue=EPI["store"], out_f32=1)
    _close(Cf, A.float() @ B.float(), 1e-5)


@pytest.mark.parametrize("simt", BACKENDS)
@pytest.mark.parametrize("K", [300, 64, 1000])
def test_wgrad_both_mn_major_ragged_k(rv, simt, K):
    M, N = 256, 384
    A, B = _bf((K, M + 128), 5), _bf((K, N + 128), 6)   # operands are column windows of wider buffers
    ref = A[:, 128:].float().T @ B[:, 128:].float()
    Cf = torch.full((M, N), float("nan"), device="cuda", dtype=torch.float32)
    _call(rv, simt, M=M, N=N, K=K, A=A, B0=B, lda=M + 128, ldb=N + 128, a_mn_major=1, b_mn_major=1, a_col0=128,
          b_col0=128, C=Cf, ldc=N, epilogue=EPI["wgrad"])
    _close(Cf, ref, 1e-5)
    _call(rv, simt, M=M, N=N, K=K, A=A, B0=B, lda=M + 128, ldb=N + 128, a_mn_major=1, b_mn_major=1, a_col0=128,
          b_col0=128, C=Cf, ldc=N, epilogue=EPI["wgrad"], accumulate=1)
    _close(Cf, 2 * ref, 1e-5)


@pytest.mark.parametrize("simt", BACKENDS)
def test_swiglu_n_concat(rv, simt):
    M, N, K = 260, 384, 256
    A, Bg, Bu = _bf((M, K), 7), _bf((N, K), 8, 0.2), _bf((N, K), 9, 0.2)
    H = torch.full((M, N), float("nan"), device="cuda", dtype=torch.bfloat16)
    AB = torch.full((M, 2 * N), float("nan"), device="cuda", dtype=torch.bfloat16)
    _call(rv, simt, M=M, N=N, K=K, A=A, B0=Bg, B1=Bu, lda=K, ldb=K, concat=1, C=H, ldc=N, C1=AB, ldc1=2 * N,
          epilogue=EPI["swiglu"])
    a, b = A.float() @ Bg.float().T, A.float() @ Bu.float().T
    _close(H, torch.nn.functional.silu(a) * b)
    _close(AB[:, :N], a)
    _close(AB[:, N:], b)
    # without the copy of the pre-activations, and with a per-row scale on H
    rs = torch.rand(M, device="cuda") + 0.1
    H2 = torch.full((M, N), float("nan"), device="cuda", dtype=torch.bfloat16)
    _call(rv, simt, M=M, N=N, K=K, A=A, B0=Bg, B1=Bu, lda=K, ldb=K, concat=1, C=H2, ldc=N, rowscale=rs,
          epilogue=EPI["swiglu"])
    _close(H2, rs[:, None] * torch.nn.functional.silu(a) * b)
    H3 = torch.full((M, N), float("nan"), device="cuda", dtype=torch.bfloat16)
    _call(rv, simt, M=M, N=N, K=K, A=A, B0=Bg, B1=Bu, lda=K, ldb=K, concat=1, C=H3, ldc=N, C1=AB, ldc1=2 * N, rowscale=rs,
          epilogue=EPI["swiglu"])
    assert torch.equal(H3, H2)


@pytest.mark.parametrize("simt", BACKENDS)
def test_k_concat_b_mn_major(rv, simt):
    M, N, Kh = 200, 256, 384
    A, B0, B1 = _bf((M, 2 * Kh), 10), _bf((Kh, N), 11), _bf((Kh, N), 12)
    Cb = torch.full((M, N), float("nan"), device="cuda", dtype=torch.bfloat16)
    _call(rv, simt, M=M, N=N, K=2 * Kh, A=A, B0=B0, B1=B1, lda=2 * Kh, ldb=N, b_mn_major=1, concat=2, C=Cb, ldc=N,
          epilogue=EPI["store"])
    _close(Cb, A[:, :Kh].float() @ B0.float() + A[:, Kh:].float() @ B1.float())


@pytest.mark.parametrize("simt", BACKENDS)
def test_rowscale_and_couple(rv, simt):
    M, N, K = 300, 256, 128
    A, B = _bf((M, K), 13), _bf((N, K), 14)
    rs = torch.rand(M, device="cuda")
    Cb = torch.full((M, N), float("nan"), device="cuda", dtype=torch.bfloat16)
    _call(rv, simt, M=M, N=N, K=K, A=A, B0=B, lda=K, ldb=K, C=Cb, ldc=N, rowscale=rs, epilogue=EPI["rowscale"])
    ref = A.float() @ B.float().T
    _close(Cb, rs[:, None] * ref)
    # coupling epilogue on strided fp32 streams
    X = torch.randn(M, 2 * N, device="cuda")
    Y = torch.full((M, 2 * N), float("nan"), device="cuda")
    for sign in (1.0, -1.0):
        _call(rv, simt, M=M, N=N, K=K, A=A, B0=B, lda=K, ldb=K, C=Y, ldc=2 * N, resid=X, ld_resid=2 * N,
              resid_sign=sign, epilogue=EPI["couple"])
        _close(Y[:, :N], X[:, :N] + sign * ref, 1e-5)
        assert torch.isnan(Y[:, N:]).all()


@pytest.mark.parametrize("simt", BACKENDS)
def test_dswiglu(rv, simt):
    M, N, K = 300, 256, 128
    A, B = _bf((M, K), 15), _bf((K, N), 16, 0.3)
    AB = _bf((M, 2 * N), 17)
    AB0 = AB.clone()
    rs = torch.rand(M, device="cuda") + 0.1
    parts = N // 64 if simt else 2 * ((N + 255) // 256)      # partials per row
    dg = torch.full((M, parts), float("nan"), device="cuda")
    _call(rv, simt, M=M, N=N, K=K, A=A, B0=B, lda=K, ldb=N, b_mn_major=1, ab=AB, ld_ab=2 * N, rowscale=rs,
          dg_part=dg, dg_ld=parts, epilogue=EPI["dswiglu"])
    acc = A.float() @ B.float()
    a, b = AB0[:, :N].float(), AB0[:, N:].float()
    s = torch.sigmoid(a)
    H = a * s * b
    dH = rs[:, None] * acc
    _close(AB[:, :N], dH * b * (s * (1 + a * (1 - s))))
    _close(AB[:, N:], dH * a * s)
    _close(dg.sum(1), (acc * H).sum(1), 1e-3)


def _groups(counts):
    off = [0]
    for c in counts:
        off.append(off[-1] + ((c + 127) // 128) * 128)
    tile_group = []
    for e in range(len(counts)):
        tile_group += [e] * ((off[e + 1] - off[e]) // 128)
    return off, tile_group


@pytest.mark.parametrize("simt", BACKENDS)
def test_grouped_rows_and_grouped_k(rv, simt):
    counts = [130, 0, 5, 256, 1]
    E = len(counts)
    off, tile_group = _groups(counts)
    rows = off[-1]
    rows_cap = rows + 256                              # buffers are sized for an upper bound
    N, K = 256, 128
    A = torch.zeros(rows_cap, K, device="cuda", dtype=torch.bfloat16)
    for e, c in enumerate(counts):
        A[off[e]: off[e] + c] = _bf((c, K), 20 + e)
    A[rows:] = float("nan")                            # never read
    W = _bf((E, N, K), 30)
    g_off = torch.tensor(off, dtype=torch.int32, device="cuda")
    g_tile = torch.tensor(tile_group + [0] * 8, dtype=torch.int32, device="cuda")
    g_total = torch.tensor([rows], dtype=torch.int32, device="cuda")
    Cb = torch.full((rows_cap, N), 7.0, device="cuda", dtype=torch.bfloat16)
    _call(rv, simt, M=rows_cap, N=N, K=K, A=A, B0=W, lda=K, ldb=K, C=Cb, ldc=N, epilogue=EPI["store"], group_mode=1,
          n_groups=E, group_off=g_off, tile_group=g_tile, rows_total=g_total, b_group_stride=N * K)
    for e, c in enumerate(counts):
        if c:
            _close(Cb[off[e]: off[e] + c], A[off[e]: off[e] + c].float() @ W[e].float().T)
        assert (Cb[off[e] + c: off[e + 1]] == 0).all()                    # padding rows come out as zeros
    assert (Cb[rows:] == 7.0).all()                                       # rows past the total are untouched
    # grouped K: per-expert weight gradient  dW[e] = A_e^T B_e
    Bm = torch.zeros(rows_cap, N, device="cuda", dtype=torch.bfloat16)
    Bm[:rows] = _bf((rows, N), 40)
    for e, c in enumerate(counts):
        Bm[off[e] + c: off[e + 1]] = 0
    Am = A.clone(); Am[rows:] = 0
    dW = torch.full((E, K, N), float("nan"), device="cuda")
    _call(rv, simt, M=K, N=N, K=rows_cap, A=Am, B0=Bm, lda=K, ldb=N, a_mn_major=1, b_mn_major=1, C=dW, ldc=N,
          epilogue=EPI["wgrad"], group_mode=2, n_groups=E, group_off=g_off, c_group_stride=K * N)
    for e, c in enumerate(counts):
        ref = Am[off[e]: off[e + 1]].float().T @ Bm[off[e]: off[e + 1]].float()
        if c == 0:
            assert (dW[e] == 0).all()
        else:
            _close(dW[e], ref, 1e-5)


def _chunks(counts, off):
    out = []
    for e, c in enumerate(counts):
        n = ((c + 31) // 32) * 32
        for r in range(0, n, 256):
            out.append([e, off[e] + r, min(256, n - r), 0])
    return out


@pytest.mark.parametrize("counts", [[130, 0, 5, 256, 1], [700, 33, 0, 257, 64, 1000], [0, 0, 3]])
def test_grouped_rows_with_tokens_on_the_mma_n_side(rv, counts):
    """The transposed pair mode of the tcgen05 back end (weights on M, an expert's real rows on N) against the
    plain evaluation and against the row-tiled mode of the same kernel: store, gate scale, K concatenation
    with [K, N] weights."""
    E = len(counts)
    off, tile_group = _groups(counts)
    rows = off[-1]
    rows_cap = rows + 256
    N, K = 512, 192
    A = torch.zeros(rows_cap, K, device="cuda", dtype=torch.bfloat16)
    for e, c in enumerate(counts):
        A[off[e]: off[e] + c] = _bf((c, K), 20 + e)
    W = _bf((E, N, K), 30)
    ch = _chunks(counts, off)
    g_off = torch.tensor(off, dtype=torch.int32, device="cuda")
    g_tile = torch.tensor(tile_group + [0] * 8, dtype=torch.int32, device="cuda")
    g_total = torch.tensor([rows, len(ch)], dtype=torch.int32, device="cuda")
    g_ch = torch.tensor(ch + [[0, 0, 0, 0]], dtype=torch.int32, device="cuda")
    scale = torch.zeros(rows_cap, device="cuda")
    for e, c in enumerate(counts):
        scale[off[e]: off[e] + c] = torch.rand(c, device="cuda") + 0.5
    common = dict(M=rows_cap, N=N, K=K, A=A, B0=W, lda=K, ldb=K, ldc=N, group_mode=1, n_groups=E, group_off=g_off,
                  tile_group=g_tile, rows_total=g_total, b_group_stride=N * K)
    for epi in ("store", "rowscale"):
        Ct = torch.full((rows_cap, N), 7.0, device="cuda", dtype=torch.bfloat16)
        Cr = torch.full((rows_cap, N), 7.0, device="cuda", dtype=torch.bfloat16)
        _call(rv, False, C=Ct, epilogue=EPI[epi], rowscale=scale, tok_chunks=g_ch, **common)
        _call(rv, False, C=Cr, epilogue=EPI[epi], rowscale=scale, **common)
        for e, c in enumerate(counts):
            if c:
                ref = A[off[e]: off[e] + c].float() @ W[e].float().T
                if epi == "rowscale":
                    ref = ref * scale[off[e]: off[e] + c, None]
                _close(Ct[off[e]: off[e] + c], ref)
                assert torch.equal(Ct[off[e]: off[e] + c], Cr[off[e]: off[e] + c])      # same products, same rounding
            n32 = ((c + 31) // 32) * 32
            assert (Ct[off[e] + c: off[e] + n32] == 0).all()       # rows up to the next multiple of 32: zeros
            assert (Ct[off[e] + n32: off[e + 1]] == 7.0).all()     # further padding rows are not touched in this mode
        assert (Ct[rows:] == 7.0).all()
    # K concatenation with weights stored [K, N] (the shape of dU = da Wg + db Wu)
    Kh = 128
    A2 = torch.zeros(rows_cap, 2 * Kh, device="cuda", dtype=torch.bfloat16)
    for e, c in enumerate(counts):
        A2[off[e]: off[e] + c] = _bf((c, 2 * Kh), 50 + e)
    W0, W1 = _bf((E, Kh, N), 60, 0.3), _bf((E, Kh, N), 61, 0.3)
    Ct = torch.zeros(rows_cap, N, device="cuda", dtype=torch.bfloat16)
    _call(rv, False, M=rows_cap, N=N, K=2 * Kh, A=A2, B0=W0, B1=W1, lda=2 * Kh, ldb=N, b_mn_major=1, concat=2, C=Ct, ldc=N,
          epilogue=EPI["store"], group_mode=1, n_groups=E, group_off=g_off, tile_group=g_tile, rows_total=g_total,
          b_group_stride=Kh * N, tok_chunks=g_ch)
    for e, c in enumerate(counts):
        if c:
            a = A2[off[e]: off[e] + c].float()
            _close(Ct[off[e]: off[e] + c], a[:, :Kh] @ W0[e].float() + a[:, Kh:] @ W1[e].float())


def test_load_forms_give_the_same_bits(rv):
    """The operand loads have two switches that must not change a result: one or two load threads, and MN-major
    operands through 3-D tensor maps (128 columns per load) or through 64 x 64 boxes of 2-D maps (the form the
    library falls back to when a leading dimension is not a multiple of 64).  Every product shape with an
    MN-major operand, in all four combinations, against the default."""
    counts = [130, 0, 5, 300, 64]
    E = len(counts)
    off, tile_group = _groups(counts)
    rows = off[-1]
    ch = _chunks(counts, off)
    g_off = torch.tensor(off, dtype=torch.int32, device="cuda")
    g_tile = torch.tensor(tile_group + [0] * 8, dtype=torch.int32, device="cuda")
    g_total = torch.tensor([rows, len(ch)], dtype=torch.int32, device="cuda")
    g_ch = torch.tensor(ch + [[0, 0, 0, 0]], dtype=torch.int32, device="cuda")
    K, N = 256, 384                                     # N = 384: the last column tile is 128 wide
    X = torch.zeros(rows, K, device="cuda", dtype=torch.bfloat16)
    for e, c in enumerate(counts):
        X[off[e]: off[e] + c] = _bf((c, K), 70 + e)
    Wkn = _bf((E, K, N), 80, 0.3)                       # weights stored [K, N]
    G = torch.zeros(rows, N, device="cuda", dtype=torch.bfloat16)
    for e, c in enumerate(counts):
        G[off[e]: off[e] + c] = _bf((c, N), 90 + e)
    Kh = 128
    W0, W1 = _bf((E, Kh, N), 60, 0.3), _bf((E, Kh, N), 61, 0.3)
    Ad, Bd = _bf((1000, 256 + 128), 5), _bf((1000, N + 128), 6)

    def products(**dbg):
        out = {}
        # row-tiled experts, B [K, N] (the shape of dH = dO W_down)
        out["rows"] = torch.zeros(rows, N, device="cuda", dtype=torch.bfloat16)
        _call(rv, False, M=rows, N=N, K=K, A=X, B0=Wkn, lda=K, ldb=N, b_mn_major=1, C=out["rows"], ldc=N, epilogue=EPI["store"],
              group_mode=1, n_groups=E, group_off=g_off, tile_group=g_tile, rows_total=g_total, b_group_stride=K * N, **dbg)
        # transposed pair mode, K concatenation of two [K, N] weights (the shape of dU = da W_g + db W_u)
        out["tr"] = torch.zeros(rows, N, device="cuda", dtype=torch.bfloat16)
        _call(rv, False, M=rows, N=N, K=2 * Kh, A=X, B0=W0, B1=W1, lda=K, ldb=N, b_mn_major=1, concat=2, C=out["tr"], ldc=N,
              epilogue=EPI["store"], group_mode=1, n_groups=E, group_off=g_off, tile_group=g_tile, rows_total=g_total,
              b_group_stride=Kh * N, tok_chunks=g_ch, **dbg)
        # K-grouped weight gradient, both operands MN-major
        out["wgrad"] = torch.zeros(E, K, N, device="cuda")
        _call(rv, False, M=K, N=N, K=rows, A=X, B0=G, lda=K, ldb=N, a_mn_major=1, b_mn_major=1, C=out["wgrad"], ldc=N,
              epilogue=EPI["wgrad"], group_mode=2, n_groups=E, group_off=g_off, c_group_stride=K * N, **dbg)
        # dense weight gradient from column windows of wider buffers, ragged K
        out["dense"] = torch.zeros(256, N, device="cuda")
        _call(rv, False, M=256, N=N, K=1000, A=Ad, B0=Bd, lda=256 + 128, ldb=N + 128, a_mn_major=1, b_mn_major=1, a_col0=128,
              b_col0=128, C=out["dense"], ldc=N, epilogue=EPI["wgrad"], **dbg)
        # dense product with B [K, N]
        out["store"] = torch.zeros(1000, N, device="cuda", dtype=torch.bfloat16)
        _call(rv, False, M=1000, N=N, K=256 + 128, A=Ad, B0=Wkn[0].contiguous().repeat(2, 1)[:256 + 128].contiguous(), lda=256 + 128,
              ldb=N, b_mn_major=1, C=out["store"], ldc=N, epilogue=EPI["store"], **dbg)
        return out

    ref = products()
    _close(ref["dense"], Ad[:, 128:].float().T @ Bd[:, 128:].float(), 1e-5)
    for e, c in enumerate(counts):
        if c:
            _close(ref["rows"][off[e]: off[e] + c], X[off[e]: off[e] + c].float() @ Wkn[e].float())
    for split in (1, 2):
        for boxes in (0, 1):
            got = products(split_loads=split, mn_boxes=boxes)
            for n in ref:
                assert torch.equal(got[n], ref[n]), (n, split, boxes)
