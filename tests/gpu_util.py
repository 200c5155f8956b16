"""Helpers for the GPU parity tests: run the CUDA path through the C ABI and compare
it element by element with the fp64 oracle on the same seeded inputs."""
import numpy as np
import torch

from oracle import ref
from paper_2211_05102_b200 import binding

TOL = 2e-3   # |gpu - ref| <= TOL * (1 + |ref|), the tolerance the metric states
CANARY = 1.2345e33


def run_gpu(q, k, v, lengths, scale, plan=None, workspace=None, check_canaries=True):
    """q,k,v,lengths: CPU tensors. Returns the fp32 output as a CPU tensor."""
    B, H, D = q.shape
    Lmax = k.shape[1]
    dev = torch.device("cuda:0")
    qd, kd, vd, ld = q.to(dev), k.to(dev), v.to(dev), lengths.to(dev)
    n = B * H * D
    guard = 1024
    buf = torch.full((n + 2 * guard,), CANARY, dtype=torch.float32, device=dev)
    out = buf[guard:guard + n].view(B, H, D)
    if workspace is None:
        workspace = binding.alloc_workspace(B, H, D, Lmax)
    binding.mqa_decode(qd, kd, vd, ld, out, scale, workspace, plan=plan)
    status = binding.mqa_check_status(workspace)
    assert status == binding.MQA_OK, binding.status_string(status)
    torch.cuda.synchronize()
    if check_canaries:
        assert bool((buf[:guard] == CANARY).all()) and bool((buf[guard + n:] == CANARY).all()), "wrote outside out"
    return out.cpu().clone()


def assert_close(gpu: torch.Tensor, expect: np.ndarray, what=""):
    g = gpu.double().numpy()
    assert np.isfinite(g).all(), f"{what}: non-finite output"
    ratio = np.abs(g - expect) / (TOL * (1.0 + np.abs(expect)))
    worst = float(ratio.max()) if ratio.size else 0.0
    assert worst <= 1.0, f"{what}: max err/tol = {worst:.3f} at {np.unravel_index(ratio.argmax(), ratio.shape)}"
    return worst


def check(q, k, v, lengths, scale, plan=None, what=""):
    expect = ref.mqa_decode_ref(q, k, v, lengths, scale)
    got = run_gpu(q, k, v, lengths, scale, plan=plan)
    return assert_close(got, expect, what)


def plans_for(B, H, D, Lmax, ctas=(None,)):
    """All (path, num_ctas) plans to exercise for a shape; None = the heuristic's count."""
    out = []
    for path in (binding.MQA_PATH_FMA, binding.MQA_PATH_TC):
        try:
            base = binding.mqa_decode_plan(B, H, D, Lmax, path)
        except binding.MqaError:
            continue
        for c in ctas:
            # None: the library's own plan (adaptive block count); a number pins the block count
            out.append(base if c is None else binding.Plan(base.path, c, base.tile_rows))
    return out
