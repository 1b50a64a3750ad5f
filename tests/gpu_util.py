"""Helpers shared by the GPU parity tests: tensor conversion and the error metrics of the contract."""
import numpy as np
import torch

from spa_workloads import bf16_round

TOL = {
    # max-abs, relative RMS (None = not checked) per storage dtype
    # lse: bound when the attention call reads the same qkv bits as the oracle; lse_chain: bound in an
    # end-to-end chain, where the device qkv carries one storage rounding the oracle's does not
    # (|dS| <= scale * sum_e |dq_e k_e + q_e dk_e| with relative steps of 2^-9 in bf16).
    "f32": dict(max_abs=1e-4, rel_rms=None, lse=1e-5, lse_chain=1e-5, score=1e-4),
    "bf16": dict(max_abs=3e-2, rel_rms=1e-2, lse=1e-3, lse_chain=3e-2, score=1e-4),
}


def round_to(a, dtype):
    """fp64 array rounded to the storage dtype, as fp64 (what the next GPU call will read)."""
    a = np.asarray(a, np.float64)
    return bf16_round(a) if dtype == "bf16" else a.astype(np.float32).astype(np.float64)


def dev(a, dtype, device="cuda"):
    """fp64 numpy -> device tensor in the storage dtype."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    if dtype == "bf16":
        t = t.to(torch.bfloat16)
    return t.to(device).contiguous()


def host(t):
    return t.detach().to("cpu", torch.float64).numpy()


def errors(got, ref):
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    if ref.size == 0:
        return 0.0, 0.0
    diff = got - ref
    max_abs = float(np.abs(diff).max())
    denom = float(np.sqrt((ref ** 2).mean()))
    rel_rms = float(np.sqrt((diff ** 2).mean()) / denom) if denom > 0 else float(np.sqrt((diff ** 2).mean()))
    return max_abs, rel_rms


def assert_close(got, ref, dtype, what, scale_max_abs=False):
    """The parity bar: fp32 max-abs <= 1e-4; bf16 max-abs <= 3e-2 and relative RMS <= 1e-2.
    With scale_max_abs the max-abs bound grows with the reference magnitude (fp32 gradient sums
    whose values are far above 1, where one bf16 rounding of an input already exceeds 3e-2)."""
    assert np.all(np.isfinite(got)), f"{what}: non-finite values"
    max_abs, rel_rms = errors(got, ref)
    tol = TOL[dtype]
    bound = tol["max_abs"]
    if scale_max_abs and np.asarray(ref).size:
        bound *= max(1.0, float(np.abs(ref).max()))
        # shown with `pytest -s`: which tensors need the scaled bound, and by how much
        print(f"{what}: max-abs {max_abs:.3e} (flat bound {tol['max_abs']:.1e}, scaled bound {bound:.3e}, "
              f"max |ref| {float(np.abs(ref).max()):.3e}), rel-rms {rel_rms:.3e}")
    assert max_abs <= bound, f"{what}: max-abs {max_abs:.3e} > {bound:.3e} (rel-rms {rel_rms:.3e})"
    if tol["rel_rms"] is not None:
        assert rel_rms <= tol["rel_rms"], f"{what}: rel-rms {rel_rms:.3e} > {tol['rel_rms']:.1e}"
    return max_abs, rel_rms
