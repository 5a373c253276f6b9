"""The two product engines against a plain PyTorch fp32 product of the same (rounded) inputs."""
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2609_21102_b200 import binding
    c = binding.Context(0)
    yield c
    c.close()


def _ref(A, B, ta, tb, alpha=1.0):
    a = A.float().transpose(1, 2) if ta else A.float()
    b = B.float().transpose(1, 2) if tb else B.float()
    return alpha * torch.matmul(a.double(), b.double()).float()


def _mk(b, r, c, dtype, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return torch.randn((b, r, c), generator=g, device="cuda", dtype=torch.float32).to(dtype)


SHAPES = [(1, 128, 128, 64), (2, 200, 136, 96), (3, 256, 264, 200), (1, 72, 48, 40), (2, 384, 160, 320)]


@pytest.mark.parametrize("b,M,N,K", SHAPES)
@pytest.mark.parametrize("ta,tb", [(False, True), (False, False), (True, False), (True, True)])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_simt_engine(ctx, b, M, N, K, ta, tb, dtype):
    from paper_2609_21102_b200 import binding
    A = _mk(b, K if ta else M, M if ta else K, dtype, 1)
    B = _mk(b, N if tb else K, K if tb else N, dtype, 2)
    C = ctx.defl_debug_gemm(A, B, ta, tb, engine=binding.ENGINE_SIMT, out_dtype=torch.float32, alpha=0.5)
    ref = _ref(A, B, ta, tb, 0.5)
    assert torch.allclose(C, ref, rtol=1e-4, atol=1e-3)


@pytest.mark.parametrize("b,M,N,K", SHAPES)
@pytest.mark.parametrize("ta,tb", [(False, True), (False, False), (True, False), (True, True)])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_tensor_engine(ctx, b, M, N, K, ta, tb, dtype):
    from paper_2609_21102_b200 import binding
    A = _mk(b, K if ta else M, M if ta else K, dtype, 3)
    B = _mk(b, N if tb else K, K if tb else N, dtype, 4)
    if dtype == torch.float32 and (ta or not tb):
        # tf32 tiles are K-major only: the engine must refuse, not compute something else
        with pytest.raises(binding.DeflError) as e:
            ctx.defl_debug_gemm(A, B, ta, tb, engine=binding.ENGINE_TENSOR, out_dtype=torch.float32)
        assert e.value.code == -4
        return
    C = ctx.defl_debug_gemm(A, B, ta, tb, engine=binding.ENGINE_TENSOR, out_dtype=torch.float32)
    torch.cuda.synchronize()
    ref = _ref(A, B, ta, tb)
    if dtype == torch.bfloat16:      # exact products of bf16 values, fp32 accumulation
        assert torch.allclose(C, ref, rtol=1e-4, atol=2e-3)
    else:                            # tf32 operands: 10-bit mantissas
        err = (C - ref).norm() / ref.norm()
        assert err < 2e-3, float(err)


def test_tensor_engine_bf16_output_and_large_tiles(ctx):
    from paper_2609_21102_b200 import binding
    A = _mk(2, 520, 1600, torch.bfloat16, 5)     # X X^T with a ragged 1600 = 12.5 tiles of 128
    C = ctx.defl_debug_gemm(A, A, False, True, engine=binding.ENGINE_TENSOR, out_dtype=torch.bfloat16)
    ref = _ref(A, A, False, True)
    err = (C.float() - ref).norm() / ref.norm()
    assert err < 4e-3, float(err)
    B = _mk(2, 1600, 1608, torch.bfloat16, 6)    # MN-major right operand, N = 1608 ragged
    A2 = _mk(2, 264, 1600, torch.bfloat16, 7)
    C2 = ctx.defl_debug_gemm(A2, B, False, False, engine=binding.ENGINE_TENSOR, out_dtype=torch.bfloat16)
    ref2 = _ref(A2, B, False, False)
    err2 = (C2.float() - ref2).norm() / ref2.norm()
    assert err2 < 4e-3, float(err2)


@pytest.mark.parametrize("b,M,N,K", [(2, 640, 200, 200), (1, 392, 136, 96), (2, 264, 72, 320), (1, 1600, 1600, 64)])
@pytest.mark.parametrize("ta,tb", [(True, True), (False, True), (True, False)])
@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
def test_tensor_engine_transposed_output(ctx, b, M, N, K, ta, tb, out_dtype):
    """The product written transposed (the form the filter uses for X <- B X on a wide X): complete blocks take
    the coalesced path, ragged rows and columns the general one."""
    from paper_2609_21102_b200 import binding
    A = _mk(b, K if ta else M, M if ta else K, torch.bfloat16, 21)
    B = _mk(b, N if tb else K, K if tb else N, torch.bfloat16, 22)
    C = ctx.defl_debug_gemm(A, B, ta, tb, engine=binding.ENGINE_TENSOR, out_dtype=out_dtype, alpha=0.25, transpose_out=True)
    torch.cuda.synchronize()
    assert C.shape == (b, N, M)
    ref = _ref(A, B, ta, tb, 0.25).transpose(1, 2)
    if out_dtype == torch.float32:
        assert torch.allclose(C, ref, rtol=1e-4, atol=2e-3)
    else:
        assert torch.equal(C, ref.to(torch.bfloat16)) or float((C.float() - ref).norm() / ref.norm()) < 3e-3
    with pytest.raises(binding.DeflError) as e:      # the fp32 engine does not write transposed: refused, not ignored
        ctx.defl_debug_gemm(A, B, ta, tb, engine=binding.ENGINE_SIMT, out_dtype=out_dtype, transpose_out=True)
    assert e.value.code == -4


@pytest.mark.parametrize("engine_name", ["simt", "tensor"])
def test_symmetric_mirroring(ctx, engine_name):
    from paper_2609_21102_b200 import binding
    engine = binding.ENGINE_SIMT if engine_name == "simt" else binding.ENGINE_TENSOR
    A = _mk(2, 456, 320, torch.bfloat16, 8)
    C = ctx.defl_debug_gemm(A, A, False, True, engine=engine, out_dtype=torch.float32, exploit_symmetry=True)
    ref = _ref(A, A, False, True)
    assert torch.allclose(C, ref, rtol=1e-4, atol=2e-3)
    assert torch.equal(C, C.transpose(1, 2))


@pytest.mark.parametrize("knobs", [{"DEFL_TC_PAIR": "0"}, {"DEFL_TC_KSUB": "1"}, {"DEFL_TC_TILE_M": "128"},
                                   {"DEFL_TC_STAGES": "2"}, {"DEFL_TC_DYNAMIC": "1"},
                                   {"DEFL_TC_DYNAMIC": "1", "DEFL_TC_STAGES": "2"}])
@pytest.mark.parametrize("sym", [False, True])
def test_tensor_engine_other_tile_forms(monkeypatch, knobs, sym):
    """The tile forms the default rules do not pick for these shapes (single-CTA 256-row tile, one K block per
    stage, 128-row tiles, the shallowest pipeline) stay correct: a context reads the knobs when it is created."""
    from paper_2609_21102_b200 import binding
    for k, v in knobs.items():
        monkeypatch.setenv(k, v)
    ctx = binding.Context(0)
    A = _mk(2, 712, 1096, torch.bfloat16, 9)          # ragged in M (712 = 2 x 256 + 200), K = 17.1 blocks
    if sym:
        C = ctx.defl_debug_gemm(A, A, False, True, engine=binding.ENGINE_TENSOR, out_dtype=torch.float32,
                                exploit_symmetry=True)
        ref = _ref(A, A, False, True)
        assert torch.equal(C, C.transpose(1, 2))
    else:
        B = _mk(2, 1096, 328, torch.bfloat16, 10)     # MN-major right operand, ragged N
        C = ctx.defl_debug_gemm(A, B, False, False, engine=binding.ENGINE_TENSOR, out_dtype=torch.float32)
        ref = _ref(A, B, False, False)
    assert torch.allclose(C, ref, rtol=1e-4, atol=4e-3)


@pytest.mark.parametrize("K", [64, 200, 1096])
@pytest.mark.parametrize("sym", [False, True])
def test_tensor_engine_dynamic_tiles(monkeypatch, K, sym):
    """Tiles handed out through the counter (DEFL_TC_DYNAMIC), more tiles than CTA pairs so that every pair draws
    several; a one-step K, a short and a long one. Run twice: the counter must be back at zero after a launch."""
    from paper_2609_21102_b200 import binding
    monkeypatch.setenv("DEFL_TC_DYNAMIC", "1")
    ctx = binding.Context(0)
    A = _mk(14, 1000, K, torch.bfloat16, 31)
    B = A if sym else _mk(14, 1032, K, torch.bfloat16, 32)
    ref = _ref(A, B, False, True)
    for _ in range(2):
        C = ctx.defl_debug_gemm(A, B, False, True, engine=binding.ENGINE_TENSOR, out_dtype=torch.float32,
                                exploit_symmetry=sym)
        torch.cuda.synchronize()
        assert torch.allclose(C, ref, rtol=1e-4, atol=4e-3)


@pytest.mark.parametrize("ta,tb", [(False, True), (False, False), (True, False)])
@pytest.mark.parametrize("out_dtype", [torch.float16, torch.float32])
def test_tensor_engine_ieee_half(ctx, ta, tb, out_dtype):
    """IEEE half operands (the FP16 projection filter's type): exact products, fp32 accumulation."""
    from paper_2609_21102_b200 import binding
    b, M, N, K = 2, 328, 264, 200
    A = _mk(b, K if ta else M, M if ta else K, torch.float16, 21)
    B = _mk(b, N if tb else K, K if tb else N, torch.float16, 22)
    C = ctx.defl_debug_gemm(A, B, ta, tb, engine=binding.ENGINE_TENSOR, out_dtype=out_dtype)
    ref = _ref(A, B, ta, tb)
    if out_dtype == torch.float32:
        assert torch.allclose(C, ref, rtol=1e-4, atol=2e-3)
    else:
        assert torch.allclose(C.float(), ref, rtol=2.0 ** -10, atol=2e-3)      # one rounding to half on store
    As = _mk(b, 456, 320, torch.float16, 23)
    Cs = ctx.defl_debug_gemm(As, As, False, True, engine=binding.ENGINE_TENSOR, out_dtype=out_dtype, exploit_symmetry=True)
    assert torch.equal(Cs, Cs.transpose(1, 2))
    assert torch.allclose(Cs.float(), _ref(As, As, False, True), rtol=2.0 ** -10, atol=2e-3)
    # the fp32 FMA engine takes half operands too (it serves shapes the tensor engine cannot)
    Cf = ctx.defl_debug_gemm(A, B, ta, tb, engine=binding.ENGINE_SIMT, out_dtype=torch.float32)
    assert torch.allclose(Cf, ref, rtol=1e-4, atol=2e-3)


def test_bounded_wait_runs_out_and_is_reported(monkeypatch):
    """A device-side wait that nothing satisfies ends in a status bit and a normal return, not in a hang: one
    128 x 128 x 64 product (one CTA, one tile, one pipeline step) whose only pipeline step is never announced nor
    copied, with the wait limit at 2 ms. Nothing is in flight when the waits give up; the kernel frees its tensor
    memory and returns, the context stays usable and the next product is correct."""
    from paper_2609_21102_b200 import binding
    monkeypatch.setenv("DEFL_TC_WAIT_MS", "2")
    ctx = binding.Context(0)
    A, B = _mk(1, 128, 64, torch.bfloat16, 41), _mk(1, 128, 64, torch.bfloat16, 42)
    assert ctx.defl_device_wait_status() == 0
    ctx.defl_debug_gemm(A, B, False, True, engine=binding.ENGINE_TENSOR, out_dtype=torch.float32, withhold_first_step=True)
    assert ctx.defl_device_wait_status(clear=False) == binding.ST_DEVICE_WAIT
    assert ctx.defl_device_wait_status(clear=True) == binding.ST_DEVICE_WAIT      # sticky until cleared
    assert ctx.defl_device_wait_status() == 0
    C = ctx.defl_debug_gemm(A, B, False, True, engine=binding.ENGINE_TENSOR, out_dtype=torch.float32)
    assert torch.allclose(C, _ref(A, B, False, True), rtol=1e-4, atol=2e-3)
    assert ctx.defl_device_wait_status() == 0
    ctx.close()
