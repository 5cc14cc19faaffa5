"""Helpers for the GPU parity tests: move a generated problem to the device, run the library
through its C ABI (via the ctypes binding) and compare with the CPU oracle."""
import numpy as np
import torch

# Tolerances: fp32 inputs: loss relative 1e-5, gradients max-abs over max-norm 1e-4;
# bf16 inputs: 2e-3 and 2e-2.
TOL = {"f32": dict(loss=1e-5, grad=1e-4, lse=1e-5), "bf16": dict(loss=2e-3, grad=2e-2, lse=2e-3)}


def to_device(prob, device="cuda"):
    from paper_2101_06983_b200 import binding
    return binding.problem_tensors(prob, device)


def rel_err_scalar(got, ref):
    return abs(float(got) - float(ref)) / max(abs(float(ref)), 1e-30)


def grad_err(got, ref, floor=1e-300):
    """max_ij |got - ref| / max(max_ij |ref|, floor).  `floor` guards the degenerate cases whose
    exact gradient is identically zero (e.g. a single passage)."""
    ref = np.asarray(ref, np.float64)
    got = np.asarray(got, np.float64)
    return float(np.abs(got - ref).max() / max(np.abs(ref).max(), floor))


def grad_floor(prob):
    """1e-2 of the largest magnitude a gradient entry can have, max|row| / (B tau)."""
    big = max(float(np.abs(prob.Q).max()), float(np.abs(prob.P).max()))
    return 1e-2 * big / (prob.B * prob.tau)


def run_build(prob, device="cuda"):
    from paper_2101_06983_b200 import binding
    Q, P, pos = to_device(prob, device)
    out = binding.build_cache(Q, P, pos, prob.tau, prob.mask_mode)
    torch.cuda.synchronize()
    return out


def check_against_oracle(prob, out, ref, tol=None):
    tol = tol or TOL[prob.dtype]
    assert int(out.dev_status.item()) == 0
    # relative to the loss, or to the size of its terms when the loss itself is ~0 (N = 1)
    loss_scale = max(abs(ref["loss"]), 1e-3 * float(np.abs(ref["row_lse"]).mean()), 1e-6)
    assert abs(out.loss.item() - ref["loss"]) <= tol["loss"] * loss_scale
    lse = out.row_lse.cpu().numpy().astype(np.float64)
    assert np.abs(lse - ref["row_lse"]).max() <= tol["lse"] * max(1.0, np.abs(ref["row_lse"]).max())
    pl = out.pos_logit.cpu().numpy().astype(np.float64)
    assert np.abs(pl - ref["pos_logit"]).max() <= tol["lse"] * max(1.0, np.abs(ref["pos_logit"]).max())
    floor = grad_floor(prob)
    assert grad_err(out.dQ.cpu().numpy(), ref["dQ"], floor) <= tol["grad"]
    assert grad_err(out.dP.cpu().numpy(), ref["dP"], floor) <= tol["grad"]
