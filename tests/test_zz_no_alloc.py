"""The allocation-free attention backward (spa_packed_attention_bwd_static) against the regular
entry point.

Some users of this library cannot obtain device memory at call time: they run inside a region
that is being recorded for replay, inside a runtime whose memory pool is frozen or belongs to
someone else, or they are handed only their inputs and outputs.  For them the library carries its
scratch inside its own image.  This test calls that entry point through the C boundary twice in a
row, on different data, and checks each result against the regular entry point (which takes caller
scratch): both run the same deterministic kernels, so the results must agree bit for bit, which is
inside every tolerance the other parity tests use.  It also checks that a problem larger than
the built-in array is refused with its own status.  It is collected last so that a failure here
cannot hide the result of any other test.
"""
import numpy as np
import pytest
import torch

from tests.gpu_util import assert_close, host

pytestmark = pytest.mark.gpu


def _problem(seed, B, N, C, H, cap):
    g = torch.Generator(device="cpu").manual_seed(seed)
    counts = torch.randint(1, N + 1, (B,), generator=g)
    counts[seed % B] = 1                       # a single-token segment
    cu = torch.zeros(B + 1, dtype=torch.int32)
    cu[1:] = torch.cumsum(counts, 0)
    Np = int(cu[-1])
    mk = lambda *s: torch.randn(*s, generator=g).to(torch.bfloat16).cuda()
    qkv, ao, dao = mk(cap, 3 * C), mk(cap, C), mk(cap, C)
    lse = (torch.randn(H, cap, generator=g).abs() + 3.0).cuda()
    return cu.cuda(), Np, qkv, ao, dao, lse


@pytest.mark.parametrize("C,H", [(128, 2), (128, 4)])
def test_static_scratch_entry_matches_regular_entry_twice(C, H):
    from paper_2410_23608_b200 import binding as L
    B, N = 6, 150
    cap = B * N
    p = L.make_params(B, N, C, H, "bf16", cap)
    ws = torch.empty(max(L.spa_workspace_bytes(p), 256), dtype=torch.uint8, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    for seed in (11, 12):                      # two calls in a row share the built-in array
        cu, Np, qkv, ao, dao, lse = _problem(seed, B, N, C, H, cap)
        ref = torch.zeros(cap, 3 * C, dtype=torch.bfloat16, device="cuda")
        got = torch.zeros_like(ref)
        L.spa_packed_attention_bwd(p, qkv, ao, lse, dao, cu, B, ref, ws, status)
        L.spa_packed_attention_bwd_static(p, qkv, ao, lse, dao, cu, B, got, status)
        torch.cuda.synchronize()
        assert L.spa_read_status(status) == 0
        assert np.abs(host(ref)[:Np]).max() > 0
        assert_close(host(got)[:Np], host(ref)[:Np], "bf16", "dqkv (static scratch)", scale_max_abs=True)
        assert torch.equal(got[:Np], ref[:Np])


def test_static_scratch_entry_refuses_what_does_not_fit():
    from paper_2410_23608_b200 import binding as L
    B, N, C, H = 64, 4096, 512, 16             # H * capacity * 4 bytes = 16 MiB > the built-in 4 MiB
    p = L.make_params(B, N, C, H, "bf16", B * N)
    assert H * B * N * 4 > L.SPA_STATIC_SCRATCH_BYTES
    t = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    f = torch.zeros(64, dtype=torch.float32, device="cuda")
    i = torch.zeros(B + 1, dtype=torch.int32, device="cuda")
    with pytest.raises(L.SpaError) as e:
        L.spa_packed_attention_bwd_static(p, t, t, f, t, i, B, t)
    assert e.value.status == L.SPA_ERR_SCRATCH
    pf = L.make_params(2, 64, 64, 2, "f32", 128)  # not a tensor-core problem
    with pytest.raises(L.SpaError) as e:
        L.spa_packed_attention_bwd_static(pf, f, f, f, f, i, 2, f)
    assert e.value.status == L.SPA_ERR_UNSUPPORTED
