"""Out-of-bounds writes and clobbered inputs: every output buffer of the hot path sits between guard zones filled
with a sentinel, on ragged shapes (d not a multiple of m or of 4, rows that start off 16-byte boundaries, one-chunk
inputs), and the guards as well as the inputs must come back bit for bit.  Stands in for a memory checker."""

import pytest
import torch

from paper_2110_01595_b200 import binding, build, synth

pytestmark = pytest.mark.gpu

GUARD = 4096            # bytes on either side of a buffer (a multiple of 16: the buffers keep their alignment)
SENTINEL = 0xA5


def _guarded(n_bytes):
    """A byte buffer of n_bytes between two guard zones; returns (whole, view of the middle)."""
    pad = (n_bytes + 15) // 16 * 16
    whole = torch.full((GUARD + pad + GUARD,), SENTINEL, dtype=torch.uint8, device="cuda")
    return whole, whole[GUARD:GUARD + n_bytes]


def _guards_intact(whole, n_bytes):
    head = whole[:GUARD]
    tail = whole[GUARD + n_bytes:]
    return bool((head == SENTINEL).all()) and bool((tail == SENTINEL).all())


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


@pytest.mark.parametrize("P,s,m,r,d", [
    (8, 1, 2, 4, 4_099),        # d odd
    (15, 2, 5, 9, 100_003),     # several tiles, ragged last chunk
    (15, 1, 10, 12, 50_001),    # float64 paths, all-rows recovery
    (9, 1, 7, 9, 1_237),        # generic kernels
    (5, 1, 3, 5, 2),            # d < m: one padded chunk
    (45, 3, 1, 7, 30_001),      # m = 1, six groups
    (33, 2, 4, 8, 65_537),      # four groups, one of nine
    (40, 2, 12, 20, 3_001),     # m = 12 (generic kernels)
])
@pytest.mark.parametrize("dtype", ["f32", "f64"])
def test_outputs_stay_inside_their_buffers_and_inputs_are_not_written(P, s, m, r, d, dtype):
    if dtype == "f64" and m == 7:
        pytest.skip("no float64 kernel for m = 7")
    wl = synth.Workload("guard", P, s, m, d, "normal", 1.0, "gaussian", s, 60 + P + m)
    G = synth.make_grads(wl, "cuda")
    tdtype, eb = (torch.float64, 8) if dtype == "f64" else (torch.float32, 4)
    G = G.to(tdtype)
    G_before = G.clone()
    with binding.Plan(P, s, m, r, d, seed=9, dtype=dtype) as plan:
        d_c = plan.d_c
        coded_whole, coded_bytes = _guarded(P * d_c * eb)
        coded = coded_bytes.view(tdtype).view(P, d_c)
        plan.encode(G, coded)
        torch.cuda.synchronize()
        assert _guards_intact(coded_whole, P * d_c * eb)
        assert torch.equal(G, G_before)
        fresh = plan.encode(G)                                            # every entry was written: equal to an encode into an ordinary buffer
        assert torch.equal(coded, fresh)

        nodes = synth.byzantine_nodes(wl)
        received = coded.clone()
        if nodes:
            received[nodes] = synth.byzantine_rows(wl, coded, nodes)
        received_before = received.clone()
        agg_whole, agg_bytes = _guarded(d * eb)
        mask_whole, mask_bytes = _guarded(P)
        agg = agg_bytes.view(tdtype)
        plan.decode(received, agg, mask_bytes)
        status = plan.decode_status()
        assert status == 0, binding.strerror(status)
        assert _guards_intact(agg_whole, d * eb) and _guards_intact(mask_whole, P)
        assert torch.equal(received, received_before)
        assert mask_bytes.nonzero().flatten().tolist() == nodes
        agg2, mask2 = plan.decode(received)
        assert torch.equal(agg, agg2) and torch.equal(mask_bytes, mask2)
        ref = G.sum(dim=0, dtype=torch.float64)
        assert float((agg.double() - ref).abs().max()) <= 1e-4 * float(ref.abs().max())


def test_lsq_grads_and_row_overwrite_stay_inside_their_buffers():
    P, rows, d = 6, 40, 10_004
    g = torch.Generator(device="cuda").manual_seed(5)
    X = torch.randn((P * rows, d), device="cuda", generator=g)
    y = torch.randn(P * rows, device="cuda", generator=g)
    w = torch.randn(d, device="cuda", generator=g)
    X_before = X.clone()
    with binding.Plan(P, 1, 2, 4, d, seed=1) as plan:
        whole, view = _guarded(P * d * 4)
        grads = view.view(torch.float32).view(P, d)
        plan.lsq_grads(X, y, w, grads, rows=rows)
        torch.cuda.synchronize()
        assert _guards_intact(whole, P * d * 4) and torch.equal(X, X_before)
        want = torch.stack([X[i * rows:(i + 1) * rows].double().T @ (X[i * rows:(i + 1) * rows].double() @ w.double()
                                                                   - y[i * rows:(i + 1) * rows].double()) for i in range(P)])
        assert float((grads.double() - want).abs().max()) <= 1e-5 * float(want.abs().max())
        # the adversary's row overwrite into a guarded coded matrix
        d_c = plan.d_c
        cw, cb = _guarded(P * d_c * 4)
        coded = cb.view(torch.float32).view(P, d_c)
        plan.encode(grads.contiguous(), coded)
        idx = torch.tensor([0, P - 1], dtype=torch.int32, device="cuda")
        new_rows = torch.randn((2, d_c), device="cuda", generator=g)
        plan.overwrite_rows(coded, idx, new_rows)
        torch.cuda.synchronize()
        assert _guards_intact(cw, P * d_c * 4)
        assert torch.equal(coded[0], new_rows[0]) and torch.equal(coded[P - 1], new_rows[1])
