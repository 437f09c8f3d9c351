"""GPU parity of the GEMM operator (all epilogues that store a matrix) against a float64 product of the
same bf16 inputs."""
import numpy as np
import pytest

from paper_2602_12957_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def models():
    import torch
    from paper_2602_12957_b200 import runtime as R
    cfg = I.TINY
    w = I.make_weights(cfg, 1)
    return {0: R.DeviceModel(cfg, w, 0), 1: R.DeviceModel(cfg, w, 1)}


def _run(model, M, N, K, mode, seed):
    import torch
    from paper_2602_12957_b200 import binding as B
    rng = np.random.default_rng(seed)
    A = I.bf16_round(rng.standard_normal((M, K), dtype=np.float32))
    W = I.bf16_round(rng.standard_normal((N, K), dtype=np.float32) * 0.05)
    dev = model.device
    tA = torch.from_numpy(A).to(dev, torch.bfloat16)
    tW = torch.from_numpy(W).to(dev, torch.bfloat16)
    ref = A.astype(np.float64) @ W.astype(np.float64).T
    st = torch.cuda.current_stream().cuda_stream
    if mode == 0:
        C = torch.full((M, N), 7.0, dtype=torch.bfloat16, device=dev)
        B.check(B.hsd_op_linear(model.ctx, tA, tW, C, M, N, K, 0, st))
        got = C.float().cpu().numpy().astype(np.float64)
    elif mode == 1:
        base = rng.standard_normal((M, N), dtype=np.float32)
        C = torch.from_numpy(base.copy()).to(dev)
        B.check(B.hsd_op_linear(model.ctx, tA, tW, C, M, N, K, 1, st))
        got = C.cpu().numpy().astype(np.float64)
        ref = ref + base
    else:
        C = torch.full((M, N // 2), 7.0, dtype=torch.bfloat16, device=dev)
        B.check(B.hsd_op_linear(model.ctx, tA, tW, C, M, N, K, 2, st))
        got = C.float().cpu().numpy().astype(np.float64)
        g, u = ref[:, :N // 2], ref[:, N // 2:]
        ref = g / (1.0 + np.exp(-g)) * u
    torch.cuda.synchronize()
    return got, ref


SHAPES = [(1040, 2048, 1024), (70, 256, 256), (128, 64, 64), (1, 1024, 4096), (513, 8192, 1024), (300, 1024, 4096)]


@pytest.mark.parametrize("flags", [1, 0], ids=["simt", "tensor"])
@pytest.mark.parametrize("mode", [0, 1, 2])
@pytest.mark.parametrize("shape", SHAPES)
def test_linear_matches_float64_product(models, flags, mode, shape):
    M, N, K = shape
    if mode == 2 and N % 128:
        pytest.skip("SwiGLU needs an even split into 64-column halves")
    got, ref = _run(models[flags], M, N, K, mode, seed=M + N + K + mode)
    scale = np.abs(ref).max()
    if mode == 1:
        tol = 1e-4 * scale            # fp32 output: only accumulation order differs
    else:
        tol = 2.0 ** -8 * scale + 1e-3   # one bf16 rounding of the stored result
    err = np.abs(got - ref).max()
    assert err <= tol, f"shape {shape} mode {mode}: max err {err:.3e} > {tol:.3e}"


@pytest.mark.parametrize("flags", [1, 0], ids=["simt", "tensor"])
@pytest.mark.parametrize("rows", [1, 68, 300])
def test_lm_head_argmax_matches_float64(models, flags, rows):
    """Fused LM head: per-row argmax, its logit and the next token's logit against a float64 product."""
    import torch
    from paper_2602_12957_b200 import binding as B
    model = models[flags]
    cfg = model.cfg
    rng = np.random.default_rng(rows)
    h = I.bf16_round(rng.standard_normal((rows, cfg.d_model), dtype=np.float32))
    nxt = rng.integers(0, cfg.vocab, rows).astype(np.int32)
    nxt[0] = -1
    W = model.lm_head.float().cpu().numpy().astype(np.float64)
    z = h.astype(np.float64) @ W.T
    dev = model.device
    th = torch.from_numpy(h).to(dev, torch.bfloat16)
    tn = torch.from_numpy(nxt).to(dev)
    scratch = torch.empty(rows, dtype=torch.int64, device=dev)
    am = torch.empty(rows, dtype=torch.int32, device=dev)
    zm = torch.empty(rows, dtype=torch.float32, device=dev)
    zd = torch.empty(rows, dtype=torch.float32, device=dev)
    B.check(B.hsd_op_lm_head_argmax(model.ctx, th, rows, tn, scratch, rows * 8, am, zm, zd,
                                    torch.cuda.current_stream().cuda_stream))
    torch.cuda.synchronize()
    am, zm, zd = am.cpu().numpy(), zm.cpu().numpy(), zd.cpu().numpy()
    srt = np.sort(z, axis=1)
    gap = srt[:, -1] - srt[:, -2]
    assert np.abs(zm - srt[:, -1]).max() < 2e-3
    clear = gap > 5e-3
    assert np.array_equal(am[clear], z.argmax(1)[clear]) and clear.sum() > 0.5 * rows
    assert np.all(z[np.arange(rows), am] >= srt[:, -1] - 5e-3)
    assert np.isnan(zd[0])
    assert np.abs(zd[1:] - z[np.arange(1, rows), nxt[1:]]).max() < 2e-3 if rows > 1 else True


@pytest.mark.parametrize("shape", [(513, 8192, 128), (1323, 2048, 192), (513, 2048, 1024), (1323, 1024, 4096)])
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_linear_every_tile_width_and_k_slicing(models, mode, shape):
    """Every tile width (64/128/256 and the CTA pair) and, for the residual-add epilogue, 1 to 8 slices of K, on shapes whose last
    row tile is mostly beyond M and whose K loop is short (the epilogue, not the main loop, sets the pace, so
    several staged stores are in flight per warp).  Repeated, because a staging-buffer race shows up only sometimes."""
    import torch
    from paper_2602_12957_b200 import binding as B
    model = models[0]
    M, N, K = shape
    rng = np.random.default_rng(M + N + K)
    A = I.bf16_round(np.abs(rng.standard_normal((M, K), dtype=np.float32)) + 0.1)     # strictly positive: a zero
    W = I.bf16_round(np.abs(rng.standard_normal((N, K), dtype=np.float32)) * 0.05 + 0.01)   # output is always wrong
    dev = model.device
    tA = torch.from_numpy(A).to(dev, torch.bfloat16)
    tW = torch.from_numpy(W).to(dev, torch.bfloat16)
    ref = A.astype(np.float64) @ W.astype(np.float64).T
    if mode == 2:
        g, u = ref[:, :N // 2], ref[:, N // 2:]
        ref = g / (1.0 + np.exp(-g)) * u
    st = torch.cuda.current_stream().cuda_stream
    try:
        for bn in (64, 128, 256, 512):       # 512 = a pair of CTAs on a 256 x 256 tile
            if mode == 2 and bn == 64:
                continue
            for sp in ((1, 2, 3, 4, 8) if mode == 1 else (0,)):
                if mode == 1 and sp > 1 and (K // 64 + sp - 1) // sp * (sp - 1) >= K // 64:
                    continue
                B.check(B.hsd_debug_set_gemm_tile(model.ctx, bn, sp))
                for trial in range(3):
                    if mode == 1:
                        C = torch.full((M, N), 7.0, dtype=torch.float32, device=dev)
                    else:
                        C = torch.full((M, ref.shape[1]), 7.0, dtype=torch.bfloat16, device=dev)
                    B.check(B.hsd_op_linear(model.ctx, tA, tW, C, M, N, K, mode, st))
                    torch.cuda.synchronize()
                    got = C.float().cpu().numpy().astype(np.float64) - (7.0 if mode == 1 else 0.0)
                    tol = (1e-4 if mode == 1 else 2.0 ** -7) * np.abs(ref).max() + 1e-3
                    err = np.abs(got - ref).max()
                    assert err <= tol, f"shape {shape} mode {mode} tile {bn} slices {sp} trial {trial}: max err {err:.3e}"
    finally:
        B.hsd_debug_set_gemm_tile(model.ctx, 0, 0)
