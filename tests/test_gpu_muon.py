"""defl_muon_step_batched on the GPU against the fp64 oracle's Muon step, element by element on the same inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_21102_b200 import inputs

pytestmark = pytest.mark.gpu

LR, MU, WD, SCALE = 0.05, 0.95, 0.1, 0.8


@pytest.fixture(scope="module")
def ctx():
    from paper_2609_21102_b200 import binding
    c = binding.Context(0)
    yield c
    c.close()


def _rel(a, b):
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def _case(b, m, n, k, dtype, shape_index):
    """Momentum with a head (workload 2's recipe), a small gradient, weights of unit scale; all values are rounded
    to their storage type once, and both sides start from the rounded values."""
    Mom = inputs.workload_spiked(b, m, n, shape_index, spikes=k).to(dtype)
    Grad = (0.1 * inputs.randn((b, m, n), inputs.seed_for(2, shape_index, 5))).to(dtype)
    W = inputs.randn((b, m, n), inputs.seed_for(2, shape_index, 6)).to(torch.float32)
    Om = inputs.sketch(b, min(m, n), 2 * k, 2, shape_index)
    return W, Mom, Grad, Om


def _oracle(W, Mom, Grad, Om, k, nesterov, mode, storage, with_grad=True):
    outs, moms = [], []
    for i in range(W.shape[0]):
        w1, m1 = oracle.muon_step(W[i].double().numpy(), Mom[i].double().numpy(),
                                  Grad[i].double().numpy() if with_grad else None, LR, MU, k, 2 * k,
                                  Om[i].double().numpy(), 1, [oracle.MUON_QUINTIC] * 5, nesterov=nesterov,
                                  weight_decay=WD, scale=SCALE, storage=storage, gamma=1.01, mode=mode)
        outs.append(w1)
        moms.append(m1)
    return np.stack(outs), np.stack(moms)


@pytest.mark.parametrize("shape", [(96, 160), (160, 96)])
@pytest.mark.parametrize("nesterov", [False, True])
@pytest.mark.parametrize("mode", [0, 1])
def test_fp32_step_matches_oracle(ctx, shape, nesterov, mode):
    from paper_2609_21102_b200 import binding
    m, n = shape
    b, k = 3, 4
    W, Mom, Grad, Om = _case(b, m, n, k, torch.float32, 11)
    want_w, want_m = _oracle(W, Mom, Grad, Om, k, nesterov, mode, "f32")
    Wd, Md = W.cuda(), Mom.cuda()
    ctx.defl_muon_step_batched(Wd, Md, Grad.cuda(), LR, MU, k, k, 1, [list(binding.MUON_QUINTIC)] * 5, nesterov=nesterov,
                               weight_decay=WD, scale=SCALE, sketch=Om.cuda(), restore_mode=mode, gamma=1.01)
    keep = (1.0 - LR * WD) * W.double().numpy()
    # the update itself is compared, not W (which would hide it): fp32 tolerance of the polar path
    assert _rel(Wd.cpu().double().numpy() - keep, want_w - keep) <= 2e-3
    # fp32 fused multiply-add with mu rounded to fp32, against fp64: a few units of fp32 rounding of the two terms
    bound = 2.0 ** -22 * (MU * np.abs(Mom.double().numpy()) + np.abs(Grad.double().numpy()))
    assert np.all(np.abs(Md.cpu().double().numpy() - want_m) <= bound)


@pytest.mark.parametrize("shape", [(256, 384), (320, 256)])
@pytest.mark.parametrize("nesterov", [False, True])
def test_bf16_step_matches_oracle(ctx, shape, nesterov):
    from paper_2609_21102_b200 import binding
    m, n = shape
    b, k = 4, 8
    W, Mom, Grad, Om = _case(b, m, n, k, torch.bfloat16, 12)
    want_w, want_m = _oracle(W, Mom, Grad, Om, k, nesterov, 0, "bf16")
    Wd, Md = W.cuda(), Mom.cuda()
    ctx.defl_muon_step_batched(Wd, Md, Grad.cuda(), LR, MU, k, k, 1, [list(binding.MUON_QUINTIC)] * 5, nesterov=nesterov,
                               weight_decay=WD, scale=SCALE, sketch=Om.cuda(), gamma=1.01, exploit_symmetry=True)
    keep = (1.0 - LR * WD) * W.double().numpy()
    assert _rel(Wd.cpu().double().numpy() - keep, want_w - keep) <= 3e-2
    # the stored momentum: fp32 fused multiply-add then one rounding to bf16, against fp64 then one rounding:
    # equal except where the fp32 result lands within an fp32 rounding error of a bf16 tie
    got_m = Md.cpu().double().numpy()
    assert np.mean(got_m != want_m) < 1e-3
    # ... and then by one bf16 spacing of the result (plus the fp32 rounding of the two terms where they cancel)
    terms = MU * np.abs(Mom.double().numpy()) + np.abs(Grad.double().numpy())
    assert np.all(np.abs(got_m - want_m) <= np.abs(want_m) * 2.0 ** -6 + terms * 2.0 ** -22)


def test_fused_update_equals_filter_then_axpy(ctx):
    """The weight update rides on the last product's epilogue: it must give what the separate call gives."""
    from paper_2609_21102_b200 import binding
    b, m, n, k = 2, 256, 512, 8
    W, Mom, _, Om = _case(b, m, n, k, torch.bfloat16, 13)
    sched = [list(binding.MUON_QUINTIC)] * 5
    F = ctx.defl_polar_batched(Mom.cuda(), k, k, 1, sched, sketch=Om.cuda(), gamma=1.01).float()
    Wd, Md = W.cuda(), Mom.cuda()
    ctx.defl_muon_step_batched(Wd, Md, None, LR, MU, k, k, 1, sched, weight_decay=WD, scale=SCALE, sketch=Om.cuda(),
                               gamma=1.01)
    assert torch.equal(Md.cpu(), Mom)                                     # no gradient: momentum untouched
    keep = (1.0 - LR * WD) * W.cuda()
    want = -LR * SCALE * F
    # F was rounded to bf16 when stored by the separate call, the fused path adds the fp32 accumulator
    err = float(((Wd - keep) - want).norm() / want.norm())
    assert err <= 4e-3, err


@pytest.mark.parametrize("L", [4, 5])
def test_update_rides_on_a_paired_last_pass(ctx, L):
    """A shape that takes two filter steps per pass over X: with an even depth the weight update is the epilogue of a
    product with B_{t+1} B_t, with an odd one of a single step's product; both against the oracle's step."""
    from paper_2609_21102_b200 import binding
    b, m, n, k = 2, 128, 512, 8
    W, Mom, Grad, Om = _case(b, m, n, k, torch.bfloat16, 16)
    sched = [list(binding.MUON_QUINTIC)] * L
    outs, moms = [], []
    for i in range(b):
        w1, m1 = oracle.muon_step(W[i].double().numpy(), Mom[i].double().numpy(), Grad[i].double().numpy(), LR, MU, k, 2 * k,
                                  Om[i].double().numpy(), 1, [oracle.MUON_QUINTIC] * L, weight_decay=WD, scale=SCALE,
                                  storage="bf16", gamma=1.01)
        outs.append(w1)
    Wd, Md = W.cuda(), Mom.cuda()
    ctx.defl_muon_step_batched(Wd, Md, Grad.cuda(), LR, MU, k, k, 1, sched, weight_decay=WD, scale=SCALE, sketch=Om.cuda(),
                               gamma=1.01, exploit_symmetry=True)
    keep = (1.0 - LR * WD) * W.double().numpy()
    assert _rel(Wd.cpu().double().numpy() - keep, np.stack(outs) - keep) <= 3e-2


def test_bf16_weights(ctx):
    from paper_2609_21102_b200 import binding
    b, m, n, k = 2, 256, 256, 8
    W, Mom, Grad, Om = _case(b, m, n, k, torch.bfloat16, 14)
    sched = [list(binding.MUON_QUINTIC)] * 5
    W32, M32 = W.cuda(), Mom.cuda()
    ctx.defl_muon_step_batched(W32, M32, Grad.cuda(), LR, MU, k, k, 1, sched, sketch=Om.cuda(), gamma=1.01)
    W16, M16 = W.to(torch.bfloat16).cuda(), Mom.cuda()
    W16_start = W16.clone()
    ctx.defl_muon_step_batched(W16, M16, Grad.cuda(), LR, MU, k, k, 1, sched, sketch=Om.cuda(), gamma=1.01)
    assert torch.equal(M16, M32)
    # the same update applied to the bf16-rounded weights, rounded once on store
    want = (W16_start.float() + (W32 - W.cuda())).to(torch.bfloat16)
    assert float((W16.float() - want.float()).abs().max()) <= float(W16.float().abs().max()) * 2.0 ** -7


def test_past_the_deflation_cutoff_the_step_is_plain_muon(ctx):
    """Section 4, "Deflation cutoff": the step helper passes k = 0 after the cutoff; that step must be the oracle's
    Muon step without deflation (same filter, no range finder), before the cutoff the deflated one."""
    from paper_2609_21102_b200 import binding, grouping
    b, m, n, k = 3, 96, 160, 4
    W, Mom, Grad, Om = _case(b, m, n, k, torch.float32, 15)
    sched = [list(binding.MUON_QUINTIC)] * 5
    keep = (1.0 - LR * WD) * W.double().numpy()
    for step, k_want in ((0, k), (1, 0)):
        want_w, want_m = _oracle(W, Mom, Grad, Om, k_want, False, 0, "f32")
        Wd, Md = W.cuda(), Mom.cuda()
        # window as a count, oversampling as a count (so that the sketch has the width the oracle was given)
        grouping.muon_step_groups(ctx, {(m, n): Wd}, {(m, n): Md}, {(m, n): Grad.cuda()}, LR, MU, k, k, 1, sched,
                                  step=step, total_steps=2, cutoff=0.5, weight_decay=WD, scale=SCALE,
                                  sketch=Om.cuda() if k_want else None, gamma=1.01)
        assert _rel(Wd.cpu().double().numpy() - keep, want_w - keep) <= 2e-3, step
        assert np.allclose(Md.cpu().double().numpy(), want_m, rtol=1e-6, atol=1e-7)


def test_argument_errors(ctx):
    from paper_2609_21102_b200 import binding
    W = torch.zeros((1, 64, 64), device="cuda")
    Mom = torch.ones((1, 64, 64), device="cuda")
    with pytest.raises(binding.DeflError) as e:
        ctx.defl_muon_step_batched(W, Mom, None, LR, MU, 0, 0, 0, [list(binding.MUON_QUINTIC)], nesterov=True)
    assert e.value.code == -1
    with pytest.raises(binding.DeflError) as e:
        ctx.defl_muon_step_batched(W, Mom, None, LR, MU, 0, 0, 0, torch.zeros((0, 3)))     # no filter step to ride on
    assert e.value.code == -1
