"""The projection entry point that allocates nothing (its scratch is a fixed array inside the library's
device image) against the plan-based path, through the C-ABI.  Collected last on purpose: a run that stops
at the first failure has then already run every other test."""

import numpy as np
import pytest
import torch

from oracle import solon_oracle as so
from paper_2110_01595_b200 import binding, build, synth

pytestmark = pytest.mark.gpu


def test_project_noalloc_matches_plan_path_twice_in_a_row():
    build.build()
    wl = synth.small_variant(synth.WORKLOADS["vgg13"], 1_500_003)       # P = 45, d_c = 300_001: ragged tiles
    G = synth.make_grads(wl, "cuda")
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl.seed) as plan:
        coded = plan.encode(G)
        plan.set_fresh_projections(False)        # both paths must see the same vectors f: the plan's stay as they are
        K, d_c = plan.K, plan.d_c
        # a row pitch that is a multiple of 4 floats, as the entry point requires
        pitch = (d_c + 3) // 4 * 4
        f = torch.zeros((K, pitch), dtype=torch.float32, device="cuda")
        f[:, :d_c] = torch.from_numpy(plan.projection_vectors()).cuda()
        # everything the call needs exists before it: it must not allocate
        rho = torch.empty((K, wl.P), dtype=torch.float64, device="cuda")
        nu = torch.empty(wl.P, dtype=torch.float64, device="cuda")
        torch.cuda.synchronize()
        for attempt, received in enumerate((coded, synth.apply_attack(wl, coded)[0])):
            plan.decode(received)                                        # existing path: rho, nu of this input
            assert plan.decode_status() == 0
            want_rho, want_nu = plan.projections()
            rho.fill_(float("nan"))
            nu.fill_(float("nan"))
            status = binding.solon_project_noalloc(received, f, rho, nu)
            assert status == 0, binding.strerror(status)
            torch.cuda.synchronize()
            got_rho, got_nu = rho.cpu().numpy(), nu.cpu().numpy()
            # this entry point multiplies and adds in float64 throughout; the plan's kernel works in float32 runs of
            # eight terms: the parity tests' bound for projections applies (8 * 2^-24 of ||f|| ||R_k||)
            fn = np.sqrt((f.double() ** 2).sum(1).cpu().numpy())
            lim = fn[:, None] * np.sqrt(want_nu)[None, :]
            assert np.all(np.abs(got_rho - want_rho) <= 8 * 2.0 ** -24 * 1.01 * lim), attempt
            # nu is summed in float32 inside a lane before float64 takes over, so it depends on how the
            # columns are split among blocks: the parity tests' bound for nu applies
            assert np.allclose(got_nu, want_nu, rtol=1e-4), attempt
            # and against the oracle's float64 projections and row energies of the same matrix: this kernel keeps
            # exact float64 products and float64 sums for rho (only the order of the additions differs), and adds
            # nu in float32 inside a lane for a tile at a time
            R = received.cpu().numpy()
            o_rho, o_nu = so.project(R, f[:, :d_c].cpu().numpy()), so.row_energy(R)
            assert np.all(np.abs(got_rho - o_rho) <= 1e-12 * fn[:, None] * np.sqrt(o_nu)[None, :]), attempt
            assert np.allclose(got_nu, o_nu, rtol=1e-5), attempt


@pytest.mark.parametrize("K,P,d_c,pad", [(1, 7, 5, 3), (3, 15, 4099, 1), (4, 33, 70_001, 7), (2, 9, 1, 3), (4, 102, 2048, 0)])
def test_project_noalloc_against_the_oracle_on_odd_shapes(K, P, d_c, pad):
    """Every K, fewer columns than blocks (most blocks own no column), rows that start off 16-byte boundaries, and a
    row pitch of f larger than d_c with junk in the padding, which the kernel must ignore."""
    build.build()
    gen = torch.Generator(device="cuda").manual_seed(1234 + K + P)
    received = torch.randn((P, d_c), generator=gen, device="cuda", dtype=torch.float32)
    pitch = (d_c + pad + 3) // 4 * 4
    f = torch.full((K, pitch), 1.0e30, dtype=torch.float32, device="cuda")          # junk beyond d_c
    f[:, :d_c] = 1.0 + torch.randn((K, d_c), generator=gen, device="cuda", dtype=torch.float32)
    rho = torch.full((K, P), float("nan"), dtype=torch.float64, device="cuda")
    nu = torch.full((P,), float("nan"), dtype=torch.float64, device="cuda")
    for _ in range(2):
        status = binding.solon_project_noalloc(received, f, rho, nu)
        assert status == 0, binding.strerror(status)
    torch.cuda.synchronize()
    R, F = received.cpu().numpy(), f[:, :d_c].cpu().numpy()
    o_rho, o_nu = so.project(R, F), so.row_energy(R)
    lim = np.sqrt((F.astype(np.float64) ** 2).sum(1))[:, None] * np.sqrt(o_nu)[None, :]
    assert np.all(np.abs(rho.cpu().numpy() - o_rho) <= 1e-12 * lim)
    assert np.allclose(nu.cpu().numpy(), o_nu, rtol=1e-5)


def test_project_noalloc_rejects_oversized_problems():
    build.build()
    received = torch.zeros((200, 64), dtype=torch.float32, device="cuda")       # (K + 1) * P = 600 > 512
    f = torch.ones((2, 64), dtype=torch.float32, device="cuda")
    rho = torch.zeros((2, 200), dtype=torch.float64, device="cuda")
    nu = torch.zeros(200, dtype=torch.float64, device="cuda")
    assert binding.solon_project_noalloc(received, f, rho, nu) == binding.ERR_INVALID_ARG
    f5 = torch.ones((5, 64), dtype=torch.float32, device="cuda")                # K > 4
    rho5 = torch.zeros((5, 8), dtype=torch.float64, device="cuda")
    assert binding.solon_project_noalloc(received[:8].contiguous(), f5, rho5, nu[:8].contiguous()) == binding.ERR_INVALID_ARG
