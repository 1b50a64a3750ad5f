"""GPU tests of the row tiles that follow the segments: the map itself (every packed row in exactly one tile, whole
segments per tile, long segments cut from their first row) and the tiled attention calls against the oracle and
against the plain calls, through the C boundary."""
import numpy as np
import pytest
import torch

from oracle import spa_oracle as O
from tests.gpu_util import TOL, assert_close, dev, host, round_to

pytestmark = pytest.mark.gpu

CASES = {
    "ragged": [0, 1, 2, 63, 64, 65, 130, 0, 197, 7, 0, 128, 129, 1, 1, 1, 256, 3],
    "short": [40, 90, 5, 17, 120, 128, 60, 60, 60, 9],
    "long": [518, 58, 518, 58, 300],
    "empty_tail": [10, 0, 0, 0],
    "many": None,       # 700 segments of 1-40 rows: the kernels search the offsets in global memory
}


def offsets_of(name):
    if name == "many":
        counts = np.random.default_rng(5).integers(1, 41, size=700)
    else:
        counts = np.array(CASES[name])
    return np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)


def build_map(L, p, seg_np):
    n_seg = len(seg_np) - 1
    nbytes = L.spa_attention_tiles_bytes(p, n_seg)
    assert nbytes > 0
    tiles = torch.full((nbytes // 4,), -9, dtype=torch.int32, device="cuda")
    seg = torch.from_numpy(seg_np).cuda()
    L.spa_attention_tile_map(p, seg, n_seg, tiles)
    return seg, n_seg, tiles


@pytest.mark.parametrize("name", list(CASES))
def test_tile_map_covers_every_row_once_with_whole_segments(name):
    from paper_2410_23608_b200 import binding as L
    seg_np = offsets_of(name)
    Np = int(seg_np[-1])
    cap = ((Np + 300) // 8) * 8
    p = L.make_params(1, cap, 128, 2, "bf16", cap)
    seg, n_seg, tiles = build_map(L, p, seg_np)
    t = tiles.cpu().numpy()
    n = int(t[0])
    assert 0 < n and 2 + 2 * n <= t.size
    ent = t[2:2 + 2 * n].reshape(n, 2)
    covered = np.zeros(Np, np.int32)
    lens = np.diff(seg_np)
    for lo, hi in ent:
        assert 0 <= lo < hi <= Np and hi - lo <= 128
        covered[lo:hi] += 1
        s = int(np.searchsorted(seg_np, lo, side="right")) - 1       # segment of the first row
        if seg_np[s + 1] - seg_np[s] > 128:                          # a tile of a long segment: inside it, 128-aligned to its start
            assert hi <= seg_np[s + 1] and (lo - seg_np[s]) % 128 == 0
        else:                                                        # a group: starts and ends on segment boundaries
            assert lo in seg_np and hi in seg_np
    assert np.all(covered == 1)
    # greedy grouping: a group and the first non-empty segment after it never fit into one tile together
    short_groups = sorted((int(lo), int(hi)) for lo, hi in ent
                          if seg_np[int(np.searchsorted(seg_np, lo, side="right"))] - lo <= 128)
    for lo, hi in short_groups:
        nxt_end = seg_np[np.searchsorted(seg_np, hi, side="right")] if hi < Np else None
        if nxt_end is not None and nxt_end - hi <= 128:      # the next segment is a short one
            assert nxt_end - lo > 128
    assert lens.sum() == Np


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("C,H", [(128, 2), (128, 4)])    # head dimension 64 and 32
def test_tiled_attention_matches_the_oracle_and_the_plain_calls(name, C, H):
    from paper_2410_23608_b200 import binding as L
    dt = "bf16"
    seg_np = offsets_of(name)
    Np = int(seg_np[-1])
    cap = ((Np + 300) // 8) * 8
    p = L.make_params(1, cap, C, H, dt, cap)
    seg, n_seg, tiles = build_map(L, p, seg_np)
    rng = np.random.default_rng(len(name) + H)
    qkv_r = round_to(rng.normal(size=(Np, 3 * C)), dt)

    def padded(a, cols):
        buf = np.zeros((cap, cols))
        buf[:Np] = a
        return buf

    qkv = dev(padded(qkv_r, 3 * C), dt)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    ao = torch.zeros(cap, C, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(H, cap, dtype=torch.float32, device="cuda")
    ao_p, lse_p = torch.zeros_like(ao), torch.zeros_like(lse)
    L.spa_packed_attention_fwd_tiled(p, qkv, seg, n_seg, tiles, ao, lse, status)
    L.spa_packed_attention_fwd(p, qkv, seg, n_seg, ao_p, lse_p, status)
    ao_ref, lse_ref = O.attention_fwd(qkv_r, seg_np, H)
    assert_close(host(ao)[:Np], ao_ref, dt, "attn_out (tiled)")
    assert np.abs(host(lse)[:, :Np] - lse_ref).max() <= TOL[dt]["lse"]
    assert_close(host(ao)[:Np], host(ao_p)[:Np], dt, "tiled vs plain forward")
    assert not ao[Np:].any()                                     # rows past N_p are not written

    ao_r = round_to(ao_ref, dt)
    dao_r = round_to(rng.normal(size=(Np, C)), dt)
    lse_t = torch.zeros(H, cap, dtype=torch.float32, device="cuda")
    lse_t[:, :Np] = torch.from_numpy(lse_ref).float().cuda()
    ref = O.attention_bwd(qkv_r, ao_r, lse_t[:, :Np].double().cpu().numpy(), dao_r, seg_np, H)
    ws = torch.empty(max(L.spa_workspace_bytes(p), 256), dtype=torch.uint8, device="cuda")
    dqkv = torch.zeros(cap, 3 * C, dtype=torch.bfloat16, device="cuda")
    dqkv_p = torch.zeros_like(dqkv)
    args = (dev(padded(ao_r, C), dt), lse_t, dev(padded(dao_r, C), dt))
    L.spa_packed_attention_bwd_tiled(p, qkv, args[0], args[1], args[2], seg, n_seg, tiles, dqkv, ws, status)
    L.spa_packed_attention_bwd(p, qkv, args[0], args[1], args[2], seg, n_seg, dqkv_p, ws, status)
    torch.cuda.synchronize()
    assert L.spa_read_status(status) == 0
    assert_close(host(dqkv)[:Np], ref, dt, "dqkv (tiled)", scale_max_abs=True)
    assert_close(host(dqkv)[:Np], host(dqkv_p)[:Np], dt, "tiled vs plain backward", scale_max_abs=True)
    assert not dqkv[Np:].any()


def test_tile_map_limits():
    from paper_2410_23608_b200 import binding as L
    p = L.make_params(64, 4096, 128, 2, "bf16")
    assert L.spa_attention_tiles_bytes(p, 4096) > 0 and L.spa_attention_tiles_bytes(p, 4097) == 0
    pf = L.make_params(4, 196, 96, 3, "f32")
    assert L.spa_attention_tiles_bytes(pf, 4) == 0            # tensor-core problems only
    t = torch.zeros(64, dtype=torch.int32, device="cuda")
    with pytest.raises(L.SpaError) as e:
        L.spa_attention_tile_map(p, t, 5000, t)
    assert e.value.status == L.SPA_ERR_UNSUPPORTED
