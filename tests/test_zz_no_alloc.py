"""The allocation-free GRU entry point (collected last on purpose: if it fails, `pytest -x` has
already run everything else).

grim_gru_seq_static serves callers that cannot call the CUDA allocator once they are running - a
server whose memory pool owns the whole device, a real-time thread that may not block on the
allocator - by taking its per-call scratch from a fixed 8 MiB array inside the library.  It must give
the same result as grim_gru_seq, call after call, although all calls share that array and it still
holds the previous call's data.
"""
import numpy as np
import pytest
import torch

from oracle import bcr_oracle as orc
from workloads import generators as gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2108_11033_b200.build import build_library
    build_library()
    from paper_2108_11033_b200 import binding
    return binding


def _rel(a, b):
    a, b = a.double().cpu().numpy(), b.double().cpu().numpy()
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def test_static_scratch_gru_matches_allocating_entry_point(B):
    m = gen.gru_model(40, 256, 2, 33, bh=8, bw=32, compression=5, seed=90)
    T, H, L = m["T"], m["hidden"], 2
    hi = [B.grim_bcr_pack(l["W_ih"], l["mask_ih"], 8, 32, B.GRIM_F32, 0) for l in m["layers"]]
    hh = [B.grim_bcr_pack(l["W_hh"], l["mask_hh"], 8, 32, B.GRIM_F32, 0) for l in m["layers"]]
    g = B.grim_gru_create(hi, hh, [l["b_ih"] for l in m["layers"]], [l["b_hh"] for l in m["layers"]], 5000)
    try:
        x1 = torch.from_numpy(m["x"]).cuda()
        x2 = torch.from_numpy(gen.normal_f32((T, 40), 1.0, 91, 0)).cuda()
        h0 = torch.from_numpy(gen.normal_f32((L, H), 0.5, 92, 0)).cuda()
        for x, h in ((x1, None), (x2, h0)):  # two calls in a row on the shared scratch, different data
            y_ref = torch.empty(T, H, device="cuda")
            hT_ref = torch.empty(L, H, device="cuda")
            B.grim_gru_seq(g, x, y_ref, h0=h, hT=hT_ref)
            assert B.grim_gru_status(g) == B.GRIM_OK
            y = torch.full((T, H), float("nan"), device="cuda")
            hT = torch.full((L, H), float("nan"), device="cuda")
            # nothing may be allocated during the call: neither through torch's allocator (its running count of
            # allocations must not move; frees by Python's garbage collector do not matter) nor from the driver
            # (the device's free memory must not shrink)
            torch.cuda.synchronize()
            allocs_before = torch.cuda.memory_stats().get("allocation.all.allocated", 0)
            free_before = torch.cuda.mem_get_info()[0]
            B.grim_gru_seq_static(g, x, y, h0=h, hT=hT)
            assert B.grim_gru_status(g) == B.GRIM_OK
            assert torch.cuda.memory_stats().get("allocation.all.allocated", 0) == allocs_before
            assert torch.cuda.mem_get_info()[0] >= free_before
            assert _rel(y, y_ref) <= 1e-5 and _rel(hT, hT_ref) <= 1e-5
            # and against the CPU oracle: this entry point takes its own route through the library (one shared
            # pre-activation buffer, layers one after the other), so agreeing with the other entry point is not enough
            want_y, want_h = orc.gru_seq(m["layers"], x.cpu().numpy(), h0=None if h is None else h.cpu().numpy())
            assert _rel(y, torch.from_numpy(want_y)) <= 1e-5 and _rel(hT, torch.from_numpy(want_h)) <= 1e-5
        # a request that does not fit the 8 MiB array is refused on the host, before any launch
        big_T = 5000
        xb = torch.zeros(big_T, 40, device="cuda")
        yb = torch.zeros(big_T, H, device="cuda")
        with pytest.raises(B.GrimError) as e:
            B.grim_gru_seq_static(g, xb, yb)
        assert e.value.status == B.GRIM_ERR_UNSUPPORTED
        B.grim_gru_seq(g, xb, yb)  # the allocating entry point still takes it
        assert B.grim_gru_status(g) == B.GRIM_OK
    finally:
        B.grim_gru_destroy(g)
        for h in hi + hh:
            B.grim_bcr_destroy(h)
