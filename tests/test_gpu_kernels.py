"""Single-kernel parity: each CUDA kernel, called through the C ABI, against the oracle's definition
of the same operation on seeded inputs.  Shapes span several tiles, ragged tails and tiny cases."""
import numpy as np
import pytest
import torch

import eas_synth as S
from oracle import encoder_oracle as O

pytestmark = pytest.mark.gpu


def _bf16_exact(rng, shape, scale=1.0):
    return S.round_to_bf16((rng.standard_normal(shape) * scale).astype(np.float32))


def _dev(a):
    return torch.from_numpy(a).to("cuda", dtype=torch.bfloat16)


@pytest.mark.parametrize("M,N,K", [(784, 256, 768), (300, 512, 128), (129, 256, 64), (1, 32, 64), (257, 96, 640),
                                   (1000, 1024, 1024), (128, 3072, 256), (77, 288, 192),
                                   (300, 1024, 2048), (1000, 512, 4096)])   # the last two take the wide 256x512 tiles
@pytest.mark.parametrize("act,out_fp32", [(0, False), (1, False), (2, False), (0, True)])
def test_gemm_epilogues(M, N, K, act, out_fp32):
    import paper_2609_31551_b200 as P
    rng = np.random.Generator(np.random.PCG64(M * 7 + N * 3 + K + act))
    A, W, b = _bf16_exact(rng, (M, K)), _bf16_exact(rng, (N, K), 0.05), _bf16_exact(rng, (N,), 0.5)
    y = O.linear(O._t(A), O._t(W), O._t(b))
    resid = None
    if act == 1:
        y = O.gelu(y)
    if act == 2:
        y = O.silu(y[:, 0::2]) * y[:, 1::2]          # interleaved (gate_j, up_j) rows
    if out_fp32:
        r = rng.standard_normal((M, N)).astype(np.float32)
        resid = torch.from_numpy(r).cuda()
        y = y + O._t(r)
    out, status = P.kernel_gemm(_dev(A), _dev(W), _dev(b), act=act, out_fp32=out_fp32, resid=resid)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    got = out.double().cpu()
    # fp32 accumulation over K, then one rounding (bf16: 2^-9 relative; fp32 output: accumulation only)
    tol = (1e-5 if out_fp32 else 2.0 ** -8) * y.abs() + 2e-3 * max(1.0, float(K) ** 0.5 * 0.05)
    bad = (got - y).abs() > tol
    assert not bad.any(), f"{int(bad.sum())} of {bad.numel()} wrong, max err {(got - y).abs().max():.4e}, first bad {bad.nonzero()[:5].tolist()}"


@pytest.mark.parametrize("M,N,K", [(300, 512, 128), (1000, 1024, 1024), (77, 288, 192), (513, 1024, 2048), (700, 1536, 4096)])
def test_gemm_residual_accumulated_in_place(M, N, K):
    """fp32 residual stream updated in place (x += A W^T + b): the path the encoder's proj / fc2 GEMMs take."""
    import paper_2609_31551_b200 as P
    rng = np.random.Generator(np.random.PCG64(M + N))
    A, W, b = _bf16_exact(rng, (M, K)), _bf16_exact(rng, (N, K), 0.05), _bf16_exact(rng, (N,), 0.5)
    r = rng.standard_normal((M, N)).astype(np.float32)
    y = O.linear(O._t(A), O._t(W), O._t(b)) + O._t(r)
    x = torch.from_numpy(r).cuda()
    out, status = P.kernel_gemm(_dev(A), _dev(W), _dev(b), act=0, out_fp32=True, resid=x, out=x)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    err = (x.double().cpu() - y).abs()
    assert err.max() <= 1e-5 * float(y.abs().max()) + 2e-3 * max(1.0, float(K) ** 0.5 * 0.05), err.max()


@pytest.mark.parametrize("N,K", [(768, 512), (1024, 2048)])      # narrow 256x256 tiles; wide 256x512 tiles
def test_gemm_is_independent_of_sm_budget(N, K):
    import paper_2609_31551_b200 as P
    rng = np.random.Generator(np.random.PCG64(5))
    A, W, b = _dev(_bf16_exact(rng, (1500, K))), _dev(_bf16_exact(rng, (N, K), 0.05)), _dev(_bf16_exact(rng, (N,)))
    ref, _ = P.kernel_gemm(A, W, b, act=1)
    for budget in (1, 7, 37, 74, 111):
        out, _ = P.kernel_gemm(A, W, b, act=1, sm_budget=budget)
        assert torch.equal(out, ref), budget


@pytest.mark.parametrize("act,out_fp32", [(0, False), (1, False), (0, True)])
def test_gemm_tile_shapes_agree_bit_for_bit_with_large_distinct_biases(act, out_fp32):
    """The three tile shapes must give the same bits.  The bias is large and different in every 512-column block, the
    budget is small so that every CTA (pair) walks many tiles back to back, and the whole thing is repeated: a tile
    that picked up its neighbour's staged bias (the wide tile has a single bias slot that the next tile overwrites)
    would differ from the other shapes by whole units."""
    import paper_2609_31551_b200 as P
    rng = np.random.Generator(np.random.PCG64(91))
    M, N, K = 1300, 2048, 2048
    A, W = _dev(_bf16_exact(rng, (M, K))), _dev(_bf16_exact(rng, (N, K), 0.02))
    bias = np.repeat(np.arange(N // 256, dtype=np.float32) * 8.0 - 24.0, 256) + rng.standard_normal(N).astype(np.float32)
    b = _dev(S.round_to_bf16(bias))
    x0 = torch.from_numpy(rng.standard_normal((M, N)).astype(np.float32)).cuda() if out_fp32 else None

    def run(budget, shape):
        # the fp32 case is the residual update in place (x += A W^T + b), the only fp32 form the wide tile serves
        x = x0.clone() if out_fp32 else None
        out, st = P.kernel_gemm(A, W, b, act=act, out_fp32=out_fp32, resid=x, out=x, sm_budget=budget, tile_shape=shape)
        torch.cuda.synchronize()
        assert int(st[0]) == 0
        return out

    ref = run(2, 1)
    y = O.linear(O._t(A.float().cpu().numpy()), O._t(W.float().cpu().numpy()), O._t(b.float().cpu().numpy()))
    if act == 1:
        y = O.gelu(y)
    if out_fp32:
        y = y + x0.double().cpu()
    assert (ref.double().cpu() - y).abs().max() <= 2.0 ** -7 * float(y.abs().max())
    for shape in (2, 3):
        for budget in (2, 6, 148):
            for _ in range(3):
                assert torch.equal(run(budget, shape), ref), (shape, budget)


def test_gemm_wide_tile_is_refused_where_it_does_not_exist():
    import paper_2609_31551_b200 as P
    rng = np.random.Generator(np.random.PCG64(92))
    A, W, b = _dev(_bf16_exact(rng, (300, 256))), _dev(_bf16_exact(rng, (768, 256), 0.05)), _dev(_bf16_exact(rng, (768,)))
    with pytest.raises(P.EasError) as e:
        P.kernel_gemm(A, W, b, tile_shape=3)         # N = 768 is not a multiple of 512
    assert e.value.status == 2


@pytest.mark.parametrize("d", [256, 1024, 1280])
@pytest.mark.parametrize("kind", [0, 1, 2])
def test_norm(d, kind):
    import paper_2609_31551_b200 as P
    rng = np.random.Generator(np.random.PCG64(d + kind))
    rows = 1003
    x = (rng.standard_normal((rows, d)) * 3 + 0.7).astype(np.float32)
    g, b = _bf16_exact(rng, (d,), 0.1) + 1, _bf16_exact(rng, (d,), 0.1)
    g = S.round_to_bf16(g)
    eps = 1e-5 if kind == 0 else 1e-6
    if kind == 0:
        ref = O.layer_norm(O._t(x), O._t(g), O._t(b), eps)
    elif kind == 1:
        ref = O.rms_norm(O._t(x), O._t(g), eps)
    else:
        ref = O._t(x)
    xd = torch.from_numpy(x).cuda()
    y = P.kernel_norm(xd, _dev(g), _dev(b), kind, eps)
    y32 = P.kernel_norm(xd, _dev(g), _dev(b), kind, eps, out_fp32=True) if kind != 2 else None
    torch.cuda.synchronize()
    assert (y.double().cpu() - ref).abs().max() <= 2.0 ** -8 * ref.abs().max() + 1e-6
    if y32 is not None:
        assert (y32.double().cpu() - ref).abs().max() <= 2e-5 * max(1.0, float(ref.abs().max()))
    y2 = P.kernel_norm(xd, _dev(g), _dev(b), kind, eps, sm_budget=5)
    assert torch.equal(y, y2)


@pytest.mark.parametrize("hd,H", [(64, 3), (80, 2)])
@pytest.mark.parametrize("lens", [[5], [128], [129, 1, 64, 577], [200, 1000]])
@pytest.mark.parametrize("impl", [0, 1, 2])
def test_attention_block_diagonal(hd, H, lens, impl):
    import paper_2609_31551_b200 as P
    rng = np.random.Generator(np.random.PCG64(hd + len(lens) + sum(lens)))
    T, d = sum(lens), H * hd
    qkv = _bf16_exact(rng, (T, 3 * d))
    qkv[:, : 2 * d] *= 1.5            # sharp softmax: score std about 2
    qkv = S.round_to_bf16(qkv)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    q = O._t(qkv)
    ref = torch.cat([O.attention_one_item(q[a:b, :d].reshape(-1, H, hd), q[a:b, d:2 * d].reshape(-1, H, hd),
                                          q[a:b, 2 * d:].reshape(-1, H, hd)) for a, b in zip(cu[:-1], cu[1:])])
    out, status = P.kernel_attention(_dev(qkv), cu, H, hd, impl=impl)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    err = (out.double().cpu() - ref).abs().max()
    # P is rounded to bf16 before P*V and the output to bf16: a few 2^-9 of |v| <= ~4
    assert err <= 2e-2, err
    out2, _ = P.kernel_attention(_dev(qkv), cu, H, hd, impl=impl, sm_budget=3)
    assert torch.equal(out, out2)


@pytest.mark.parametrize("H", [1, 2, 5, 16])
def test_attention_dual_head_units(H):
    """head_dim 64, items with an odd number of 128-row query tiles: their last tiles of two adjacent heads share a
    unit (with an odd head count the last head's tile stays alone); items with an even count in the same launch keep
    the ordinary units.  The tcgen05 kernel must agree with the oracle and, bit for bit, with itself at another budget;
    the register-tile kernel (impl 1) has no such units and serves as a second opinion."""
    import paper_2609_31551_b200 as P
    hd, lens = 64, [577, 65, 640, 320, 577, 128, 1]
    rng = np.random.Generator(np.random.PCG64(900 + H))
    T, d = sum(lens), H * hd
    qkv = _bf16_exact(rng, (T, 3 * d))
    qkv[:, : 2 * d] *= 1.5
    qkv = S.round_to_bf16(qkv)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    q = O._t(qkv)
    ref = torch.cat([O.attention_one_item(q[a:b, :d].reshape(-1, H, hd), q[a:b, d:2 * d].reshape(-1, H, hd),
                                          q[a:b, 2 * d:].reshape(-1, H, hd)) for a, b in zip(cu[:-1], cu[1:])])
    out, status = P.kernel_attention(_dev(qkv), cu, H, hd, impl=0)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    err = (out.double().cpu() - ref).abs()
    assert err.max() <= 2e-2, (err.max(), np.unravel_index(int(err.argmax()), err.shape))
    for budget in (1, 7, 40):
        out2, _ = P.kernel_attention(_dev(qkv), cu, H, hd, impl=0, sm_budget=budget)
        assert torch.equal(out, out2), budget
    out3, _ = P.kernel_attention(_dev(qkv), cu, H, hd, impl=1)
    assert (out.float() - out3.float()).abs().max() <= 2e-2


@pytest.mark.parametrize("H", [1, 3])
def test_attention_head_dim_80_key_tile_edges(H):
    """head_dim 80 runs on 112-key tiles with one issuer thread per warpgroup: item lengths around the multiples of 112
    and of 128 (query tiles stay 128 rows), single-tile items whose second warpgroup idles, and few CTAs for many units
    (long per-CTA unit sequences, look-ahead across unit boundaries)."""
    import paper_2609_31551_b200 as P
    hd, lens = 80, [112, 113, 224, 225, 336, 1, 127, 128, 129, 257, 640, 1000, 16, 111]
    rng = np.random.Generator(np.random.PCG64(1200 + H))
    T, d = sum(lens), H * hd
    qkv = _bf16_exact(rng, (T, 3 * d))
    qkv[:, : 2 * d] *= 1.5
    qkv = S.round_to_bf16(qkv)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    q = O._t(qkv)
    ref = torch.cat([O.attention_one_item(q[a:b, :d].reshape(-1, H, hd), q[a:b, d:2 * d].reshape(-1, H, hd),
                                          q[a:b, 2 * d:].reshape(-1, H, hd)) for a, b in zip(cu[:-1], cu[1:])])
    out, status = P.kernel_attention(_dev(qkv), cu, H, hd, impl=0)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    err = (out.double().cpu() - ref).abs()
    assert err.max() <= 2e-2, (err.max(), np.unravel_index(int(err.argmax()), err.shape))
    for budget in (1, 2, 5, 37):
        out2, st2 = P.kernel_attention(_dev(qkv), cu, H, hd, impl=0, sm_budget=budget)
        torch.cuda.synchronize()
        assert int(st2[0]) == 0
        assert torch.equal(out, out2), budget


@pytest.mark.parametrize("hd", [64, 80])
@pytest.mark.parametrize("case", ["rising", "falling", "steep_rising", "late_spike", "peaked", "uniform", "tiny_scores"])
def test_attention_softmax_degenerate_score_patterns(hd, case):
    """The online softmax across key tiles under score patterns that stress it: scores that rise with the key index
    (the running maximum grows in every tile, every earlier partial sum is rescaled), scores that fall (the first
    tile holds the maximum, later tiles underflow), one dominant key per query with score gaps of hundreds (the
    output is that key's value row), equal keys (the output is the mean of the values: a closed form), and scores
    of magnitude 1e-3.  Two more put a score far above everything seen so far into a LATER key tile, hundreds of
    octaves above the running maximum, where 2^(score - stale maximum) overflows fp32: a ramp that climbs thousands
    per tile, and one spike key per item among small scores."""
    import paper_2609_31551_b200 as P
    H, lens = 2, [700, 130]
    T, d = sum(lens), H * hd
    rng = np.random.Generator(np.random.PCG64(77 + hd))
    q = _bf16_exact(rng, (T, d))
    k = _bf16_exact(rng, (T, d))
    v = _bf16_exact(rng, (T, d))
    pos = np.concatenate([np.arange(n) for n in lens]).astype(np.float32)[:, None]
    if case in ("rising", "falling"):
        # q = all ones, k = +-(index / 64) on every coordinate: score = +-index * hd / 64 / sqrt(hd), a ramp of
        # 0 ... 87 (hd 64) or 98 (hd 80) over 700 keys
        q[:] = 1.0
        k[:] = (pos / 64.0) * (1.0 if case == "rising" else -1.0)
    elif case == "steep_rising":
        q[:] = 1.0
        k[:] = pos * 4.0
    elif case == "late_spike":
        q[:] = 1.0
        k *= 0.125
        k[500] = 50.0                       # item 0, fourth key tile
        k[700 + 129] = 50.0                 # item 1, second key tile (its last key)
    elif case == "peaked":
        q *= 6.0
        k *= 6.0
    elif case == "uniform":
        k[:] = k[0:1]
    else:
        q *= 2.0 ** -5
        k *= 2.0 ** -5
    qkv = S.round_to_bf16(np.concatenate([q, k, v], axis=1))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    t = O._t(qkv)
    ref = torch.cat([O.attention_one_item(t[a:b, :d].reshape(-1, H, hd), t[a:b, d:2 * d].reshape(-1, H, hd),
                                          t[a:b, 2 * d:].reshape(-1, H, hd)) for a, b in zip(cu[:-1], cu[1:])])
    if case == "uniform":
        vv = torch.from_numpy(qkv[:, 2 * d:].astype(np.float64))
        want = torch.cat([vv[a:b].mean(0, keepdim=True).expand(b - a, -1) for a, b in zip(cu[:-1], cu[1:])])
        assert (ref - want).abs().max() < 1e-12                      # the oracle against the closed form
    for impl in (0, 1, 2):
        out, status = P.kernel_attention(_dev(qkv), cu, H, hd, impl=impl)
        torch.cuda.synchronize()
        assert int(status[0]) == 0
        got = out.double().cpu()
        assert torch.isfinite(got).all()
        err = (got - ref).abs().max()
        assert err <= 2e-2, (case, impl, float(err))


@pytest.mark.parametrize("act", [1, 2])
def test_gemm_activation_over_a_wide_input_range(act):
    """GELU (erf form) and SwiGLU on pre-activations from -50 to 50: the far tails (exactly x, exactly -0 / 0), the
    region around zero, and the transition in between, against the oracle's definition.  A has one non-zero per row,
    so the pre-activation of row i is exactly ramp[i] * W[:, i % K] + b."""
    import paper_2609_31551_b200 as P
    M, N, K = 1024, 256, 64
    A = np.zeros((M, K), np.float32)
    ramp = S.round_to_bf16(np.linspace(-50.0, 50.0, M).astype(np.float32))
    A[np.arange(M), np.arange(M) % K] = ramp
    rng = np.random.Generator(np.random.PCG64(act))
    W = S.round_to_bf16(np.where(rng.random((N, K)) < 0.5, 1.0, 0.5).astype(np.float32))
    b = _bf16_exact(rng, (N,), 0.25)
    y = O.linear(O._t(A), O._t(W), O._t(b))
    y = O.gelu(y) if act == 1 else O.silu(y[:, 0::2]) * y[:, 1::2]
    out, status = P.kernel_gemm(_dev(A), _dev(W), _dev(b), act=act)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    got = out.double().cpu()
    assert torch.isfinite(got).all()
    tol = 2.0 ** -8 * y.abs() + 1e-4
    bad = (got - y).abs() > tol
    assert not bad.any(), f"{int(bad.sum())} wrong, max err {(got - y).abs().max():.3e}, first {bad.nonzero()[:4].tolist()}"


@pytest.mark.parametrize("kind", [0, 1])
def test_norm_rows_with_large_offsets_and_constant_rows(kind):
    """LayerNorm / RMSNorm on rows whose mean is a thousand times their spread (a one-pass variance would cancel), on
    constant rows (variance 0: the result is beta, or gamma * x / sqrt(x^2 + eps)) and on an all-zero row."""
    import paper_2609_31551_b200 as P
    d, rows, eps = 1024, 96, 1e-6
    rng = np.random.Generator(np.random.PCG64(300 + kind))
    x = rng.standard_normal((rows, d)).astype(np.float32)
    x[:32] += 1000.0
    x[32:64] = np.linspace(-3, 3, 32, dtype=np.float32)[:, None]
    x[64] = 0.0
    g, b = _bf16_exact(rng, (d,)), _bf16_exact(rng, (d,))
    ref = O.layer_norm(O._t(x), O._t(g), O._t(b), eps) if kind == 0 else O.rms_norm(O._t(x), O._t(g), eps)
    y = P.kernel_norm(torch.from_numpy(x).cuda(), _dev(g), _dev(b), kind, eps, out_fp32=True)
    torch.cuda.synchronize()
    got = y.double().cpu()
    assert torch.isfinite(got).all()
    if kind == 0:
        # constant rows: beta, up to the rounding of the fp32 mean (one ulp of x, magnified by 1 / sqrt(eps) = 1000)
        assert (got[32:65] - O._t(b).expand(33, -1)).abs().max() <= 2e-3
    # fp32 statistics: the mean of a row around 1000 carries 1000 * 2^-24 = 6e-5 of error against a spread of 1
    assert (got - ref).abs().max() <= 5e-4 * max(1.0, float(ref.abs().max()))
