"""Shape groups of a Deflated Muon step (Appendix D, "Grouping": matrices of one shape are stacked into one batch and
the batched range finder runs once per group per optimizer step).

Host-side bookkeeping only, no arithmetic. The library takes wide matrices as they are stored
(polar(M^T) = polar(M)^T is applied logically inside the kernels), so a group is keyed by the STORED shape and
nothing is transposed or copied per step: parameters, momenta and gradients of a group live in one [b, m, n]
buffer each, and the model's own tensors are views into it.
"""
from collections import OrderedDict


def shape_groups(shapes):
    """Indices of the 2-D shapes in `shapes`, grouped by shape in order of first appearance:
    OrderedDict {(m, n): [index, ...]}. Anything that is not two-dimensional is left out."""
    groups = OrderedDict()
    for i, s in enumerate(shapes):
        s = tuple(int(x) for x in s)
        if len(s) != 2:
            continue
        groups.setdefault(s, []).append(i)
    return groups


def stack_group(tensors, indices):
    """One contiguous [b, m, n] buffer holding tensors[i] for i in indices (copied once), and the list of views
    into it, in the same order; assigning the views back to the owners makes later steps copy-free."""
    import torch
    first = tensors[indices[0]]
    buf = torch.empty((len(indices),) + tuple(first.shape), dtype=first.dtype, device=first.device)
    views = []
    for j, i in enumerate(indices):
        t = tensors[i]
        if tuple(t.shape) != tuple(first.shape) or t.dtype != first.dtype or t.device != first.device:
            raise ValueError("tensor %d does not belong to this group" % i)
        buf[j].copy_(t)
        views.append(buf[j])
    return buf, views


def deflation_active(step, total_steps, cutoff=1.0):
    """The deflation cutoff of Section 4 ("Deflation cutoff"): deflation runs during the first `cutoff` fraction of
    the `total_steps` optimizer steps (step counted from 0) and the plain filter after it; cutoff = 1 keeps it on
    throughout, cutoff = 0 is plain Muon."""
    if not 0.0 <= cutoff <= 1.0:
        raise ValueError("cutoff is a fraction of the optimizer steps")
    if step < 0 or total_steps <= 0:
        raise ValueError("step >= 0 and total_steps > 0")
    return step < cutoff * total_steps


def muon_step_groups(ctx, weights, momenta, grads, lr, mu, window, oversample, power_iters, coeff_schedule,
                     step=None, total_steps=None, cutoff=1.0, **kw):
    """One Deflated Muon step over stacked groups: weights/momenta/grads are dicts {(m, n): [b, m, n] tensor} (grads
    may hold None). `window` is the number k of leading triplets, or a ratio w in (0, 1) meaning k = ceil(w min(m, n));
    `oversample` likewise a count or a ratio delta (Section 3: r = ceil(w m), r' = r + ceil(delta m)). With `step` and
    `total_steps` the deflation cutoff applies: past it the step runs with k = 0, which is the plain Muon step (no
    range finder, no deflation pass, the same filter)."""
    import math
    if step is not None and total_steps is not None and not deflation_active(step, total_steps, cutoff):
        window = 0
    for shape, W in weights.items():
        ms = min(shape)
        k = int(math.ceil(window * ms)) if 0 < window < 1 else int(window)
        p = int(math.ceil(oversample * ms)) if 0 < oversample < 1 else int(oversample)
        ctx.defl_muon_step_batched(W, momenta[shape], grads.get(shape), lr, mu, k, p, power_iters, coeff_schedule, **kw)
