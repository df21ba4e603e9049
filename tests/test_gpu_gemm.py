"""The member-batched GEMM kernels through the C ABI against the oracle's float64 contraction:
both engines (FP32 ALUs, tcgen05 tensor cores), all three operand orientations of the training
step (forward: K-major x K-major, data gradient: K-major x MN-major, weight gradient: MN-major x
MN-major), every epilogue, shapes spanning several tiles with ragged tails."""
import numpy as np
import pytest

from oracle import pbt_oracle as O

pytestmark = pytest.mark.gpu


def _bf16_grid(a):
    return O.round_bf16(a).astype(np.float32)


def _run(pkg, torch, M, N, K, batch, a_mn, b_mn, engine, epilogue, out_bf16, dtype="bf16", shared_a=False, seed=0):
    rng = np.random.default_rng(seed)
    grid = _bf16_grid if dtype == "bf16" else (lambda x: x.astype(np.float32))
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    A = grid(rng.standard_normal((batch, M, K)))
    B = grid(rng.standard_normal((batch, N, K)))
    if shared_a:
        A[:] = A[0]
    bias = rng.standard_normal((batch, N)).astype(np.float32) if epilogue in ("bias", "bias_relu") else None
    mask = grid(rng.standard_normal((batch, M, N))) if epilogue == "mask" else None
    if mask is not None:
        mask[:, ::7, ::5] = 0.0          # exact zeros and negative zeros must block the gradient too
        mask[:, 1::7, 1::5] = -0.0
    ref = O.grouped_gemm(A, B, bias, epilogue == "bias_relu", mask)
    dev = lambda x, t: torch.from_numpy(np.ascontiguousarray(x)).cuda().to(t).contiguous()
    Ad = dev(A.transpose(0, 2, 1) if a_mn else A, tdt)
    Bd = dev(B.transpose(0, 2, 1) if b_mn else B, tdt)
    if shared_a:
        Ad = Ad[:1].contiguous()
    Cd = torch.full((batch, M, N), float("nan"), device="cuda", dtype=torch.bfloat16 if out_bf16 else torch.float32)
    status = torch.zeros(8, dtype=torch.int32, device="cuda")
    pkg.grouped_gemm(Ad, Bd, Cd, a_mn=a_mn, b_mn=b_mn,
                     bias=dev(bias, torch.float32) if bias is not None else None, relu=epilogue == "bias_relu",
                     mask=dev(mask, tdt) if mask is not None else None, engine=engine, status=status, shared_a=shared_a)
    torch.cuda.synchronize()
    assert int(status[4]) == 0, "a bounded wait expired inside the kernel"
    got = Cd.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    # fp32 accumulation of K products of O(1) terms; bf16 output adds half an ulp (2^-9) per element
    scale = np.sqrt(K)
    atol = (2e-6 * K + (2.0 ** -8 if out_bf16 else 0.0) * 4) * scale if dtype == "bf16" else 1e-5 * scale
    if out_bf16:
        np.testing.assert_allclose(got, ref, rtol=2.0 ** -7, atol=atol)
    else:
        np.testing.assert_allclose(got, ref, rtol=1e-5, atol=atol if dtype != "bf16" else 3e-6 * K)
    return got


@pytest.fixture(scope="module")
def env():
    import torch
    import paper_1711_09846_b200 as pkg
    pkg.load_library()
    return pkg, torch


ORIENT = [(False, False), (False, True), (True, True)]


@pytest.mark.parametrize("a_mn,b_mn", ORIENT)
@pytest.mark.parametrize("shape", [(128, 128, 64, 1), (256, 256, 128, 2), (384, 512, 192, 3), (200, 328, 136, 2),
                                   (512, 1024, 784, 2), (136, 264, 72, 1)])
def test_tensor_core_fp32_out(env, a_mn, b_mn, shape):
    pkg, torch = env
    M, N, K, batch = shape
    _run(pkg, torch, M, N, K, batch, a_mn, b_mn, engine=2, epilogue="none", out_bf16=False)


@pytest.mark.parametrize("a_mn,b_mn,epilogue,out_bf16", [(False, False, "bias_relu", True), (False, False, "bias", False),
                                                         (False, True, "mask", True), (True, True, "none", False)])
@pytest.mark.parametrize("shape", [(256, 384, 256, 3), (200, 328, 136, 2), (512, 2048, 512, 1)])
def test_tensor_core_epilogues(env, a_mn, b_mn, epilogue, out_bf16, shape):
    pkg, torch = env
    M, N, K, batch = shape
    _run(pkg, torch, M, N, K, batch, a_mn, b_mn, engine=2, epilogue=epilogue, out_bf16=out_bf16, seed=3)


def test_tensor_core_many_tiles_more_than_sms(env):
    pkg, torch = env
    # 4 x 4 x 12 = 192 tiles of 128 x 256 > 148 SMs: the persistent loop and both accumulator buffers cycle
    _run(pkg, torch, 512, 1024, 256, 12, False, False, engine=2, epilogue="bias_relu", out_bf16=True, seed=5)
    _run(pkg, torch, 512, 1024, 256, 12, True, True, engine=2, epilogue="none", out_bf16=False, seed=6)


def test_tensor_core_shared_operand(env):
    pkg, torch = env
    _run(pkg, torch, 256, 256, 128, 3, False, False, engine=2, epilogue="bias", out_bf16=False, shared_a=True, seed=7)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("a_mn,b_mn", ORIENT)
@pytest.mark.parametrize("shape", [(40, 72, 24, 2), (1, 10, 136, 3), (130, 2, 65, 2), (64, 64, 16, 1), (77, 129, 2, 2),
                                   (3, 200, 300, 2), (515, 2, 1024, 2), (1, 520, 1031, 2), (300, 16, 40, 1), (16, 300, 40, 1),
                                   (70, 136, 2, 2), (33, 512, 1, 3), (64, 64, 4, 1), (40, 72, 3, 2), (1030, 512, 2, 2),
                                   (45, 264, 5, 2), (512, 10, 256, 2), (10, 1024, 256, 3), (256, 10, 1024, 2), (136, 1, 512, 2),
                                   (8, 264, 72, 2), (2, 512, 1024, 2), (264, 16, 200, 1), (40, 1024, 10, 2),
                                   (100, 2304, 2, 1), (1024, 512, 1, 2), (300, 8, 4, 2),
                                   (128, 512, 256, 3), (512, 256, 128, 2), (192, 128, 48, 2),    # all tiles interior
                                   (256, 512, 64, 8), (128, 1024, 32, 8)])                      # ... and enough of them for 128-row tiles
def test_alu_engine(env, dtype, a_mn, b_mn, shape):
    pkg, torch = env
    M, N, K, batch = shape
    for ep, ob in (("none", False), ("bias_relu", dtype == "bf16"), ("mask", dtype == "bf16")):
        _run(pkg, torch, M, N, K, batch, a_mn, b_mn, engine=1, epilogue=ep, out_bf16=ob, dtype=dtype, seed=11)


@pytest.mark.parametrize("shape", [(256, 10, 1024, 3), (2048, 10, 1024, 2), (200, 16, 264, 2), (128, 5, 256, 1), (512, 72, 512, 2)])
@pytest.mark.parametrize("epilogue,out_bf16", [("bias", False), ("bias_relu", True), ("none", False)])
def test_tensor_core_narrow_outputs(env, shape, epilogue, out_bf16):
    """Fewer than 128 output columns (a ten-wide logit layer): the B rows past N are out-of-range rows of the
    tensor map and arrive as zeros."""
    pkg, torch = env
    M, N, K, batch = shape
    _run(pkg, torch, M, N, K, batch, False, False, engine=2, epilogue=epilogue, out_bf16=out_bf16, seed=23)
    _run(pkg, torch, M, N, K, batch, False, False, engine=0, epilogue=epilogue, out_bf16=out_bf16, seed=24)


def test_unsupported_shapes_are_refused_by_the_tensor_engine(env):
    pkg, torch = env
    A = torch.zeros(1, 16, 16, device="cuda", dtype=torch.bfloat16)
    Cd = torch.zeros(1, 16, 16, device="cuda", dtype=torch.float32)
    status = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(pkg.PbtError) as e:
        pkg.grouped_gemm(A, A, Cd, engine=2, status=status)
    assert e.value.code == 2


@pytest.mark.parametrize("a_mn,b_mn,epilogue,out_bf16", [(False, False, "none", False), (False, False, "bias_relu", True),
                                                         (False, True, "mask", True), (True, True, "none", False)])
@pytest.mark.parametrize("shape", [(256, 256, 64, 1), (512, 512, 256, 3), (304, 328, 136, 2), (512, 2048, 512, 2),
                                   (768, 1024, 320, 5)])
def test_tensor_core_cta_pairs(env, a_mn, b_mn, epilogue, out_bf16, shape):
    """tcgen05 cta_group::2: two CTAs of a cluster share a 256 x 256 tile (engine 3)."""
    pkg, torch = env
    M, N, K, batch = shape
    _run(pkg, torch, M, N, K, batch, a_mn, b_mn, engine=3, epilogue=epilogue, out_bf16=out_bf16, seed=17)


def test_tensor_core_cta_pairs_many_tiles(env):
    pkg, torch = env
    # 2 x 4 x 12 = 96 pair tiles on 74 CTA pairs: the persistent loop and both accumulator buffers cycle
    _run(pkg, torch, 512, 1024, 256, 12, False, False, engine=3, epilogue="bias_relu", out_bf16=True, seed=19)
    _run(pkg, torch, 512, 1024, 256, 12, False, True, engine=3, epilogue="mask", out_bf16=True, seed=20)


def test_bounded_wait_expires_with_a_status_and_leaves_the_context_usable(env):
    """Failure detection without a fault: the kernels' bounded barrier wait, run on a barrier that nothing
    signals, gives up after its poll limit, reports PBT_ERR_TIMEOUT through the status word and returns; the
    next kernels on the same stream run normally."""
    pkg, torch = env
    status = torch.zeros(8, dtype=torch.int32, device="cuda")
    pkg.selftest_bounded_wait(status, polls=2000)
    torch.cuda.synchronize()
    assert int(status[4]) == 5 and int(status[5]) == 99          # PBT_ERR_TIMEOUT, recorded by the self-test
    with pytest.raises(pkg.PbtError):
        pkg.selftest_bounded_wait(status, polls=0)
    _run(pkg, torch, 256, 256, 128, 2, False, False, engine=2, epilogue="bias_relu", out_bf16=True)
