"""The library's own random draws (attacks 2 and 5) against the oracle's
independent implementation of the same counter-based generator.

Uniform bits are integer work: bit-exact.  Normals go through float32 log,
square root and sine / cosine on the GPU and through float64 in the oracle:
compared within 1e-5 relative, with exact zeros required to be exact zeros."""

import numpy as np
import pytest
import torch

from oracle import brace_oracle as O
from paper_2501_17392_b200 import brace as B
from paper_2501_17392_b200 import build as brace_build
from paper_2501_17392_b200 import workloads as W

pytestmark = pytest.mark.gpu
REL_TOL = 1e-5


@pytest.fixture(scope="module", autouse=True)
def _built():
    brace_build.build()
    assert torch.cuda.is_available(), "these tests need a CUDA device"


def assert_close_normals(got: np.ndarray, exp: np.ndarray):
    assert np.array_equal(got == 0, exp == 0)
    assert (np.abs(got.astype(np.float64) - exp.astype(np.float64)) <= REL_TOL * np.abs(exp.astype(np.float64))).all()


@pytest.mark.parametrize("d,ld", [(1, 1), (3, 3), (4, 4), (5, 7), (1023, 1024), (10_001, 10_004), (70_002, 70_003)])
def test_uniform_draws_bit_exact(d, ld):
    for seed, rnd, first, rows in ((0, 0, 0, 1), (2501017392, 3, 5, 4), ((1 << 64) - 1, (1 << 24) - 1, 30_000, 2)):
        out = torch.full((rows, ld), -1.0, dtype=torch.float32, device="cuda")
        B.draw_matrix(B.DRAW_UNIFORM, seed, rnd, first, out, d)
        got = out.cpu().numpy()
        for i in range(rows):
            exp = O.draw_uniform(seed, rnd, first + i, d)
            assert np.array_equal(got[i, :d].view(np.uint32), exp.view(np.uint32))
        assert (got[:, d:] == -1.0).all()                      # row padding belongs to the caller


@pytest.mark.parametrize("d,ld", [(1, 1), (2, 2), (5, 7), (4096, 4096), (50_001, 50_004), (50_001, 50_003)])
def test_normal_draws_within_tolerance(d, ld):
    seed, rnd, first, rows = 424242, 17, 3, 3
    out = torch.full((rows, ld), -7.0, dtype=torch.float32, device="cuda")
    B.draw_matrix(B.DRAW_NORMAL, seed, rnd, first, out, d)
    got = out.cpu().numpy()
    for i in range(rows):
        assert_close_normals(got[i, :d], O.draw_normal(seed, rnd, first + i, d))
    assert (got[:, d:] == -7.0).all()
    # affine form: mu + sigma * z, each operation rounded to float32
    out2 = torch.empty((rows, ld), dtype=torch.float32, device="cuda")
    B.draw_matrix(B.DRAW_NORMAL, seed, rnd, first, out2, d, mu=0.01, sigma=0.1)
    z = got[:, :d]
    exp2 = (np.float32(0.01) + (np.float32(0.1) * z).astype(np.float32)).astype(np.float32)
    assert np.array_equal(out2.cpu().numpy()[:, :d].view(np.uint32), exp2.view(np.uint32))


def test_normal_draws_far_into_a_row_and_statistics():
    """One long row: the generator's block counter passes 2^20, and the sample has the moments of N(0, 1)."""
    d = 6_000_001
    out = torch.empty((1, d), dtype=torch.float32, device="cuda")
    B.draw_matrix(B.DRAW_NORMAL, 5, 1, 9, out, d)
    z = out[0]
    assert abs(float(z.mean())) < 2e-3 and abs(float(z.var()) - 1.0) < 3e-3
    start = 5_999_000
    assert_close_normals(z[start:].cpu().numpy(), O.draw_normal(5, 1, 9, d - start, start=start))
    B.draw_matrix(B.DRAW_UNIFORM, 5, 1, 9, out, d)
    assert np.array_equal(out[0, start:].cpu().numpy(), O.draw_uniform(5, 1, 9, d - start, start=start))
    assert abs(float(out[0].mean()) - 0.5) < 1e-3


def test_draw_matrix_argument_errors():
    out = torch.zeros((2, 64), dtype=torch.float32, device="cuda")
    assert B.draw_matrix_status(2, 0, 0, 0, out, 64) == B.ERR_INVALID_ARG
    assert B.draw_matrix_status(B.DRAW_NORMAL, 0, 1 << 24, 0, out, 64) == B.ERR_INVALID_ARG
    assert B.draw_matrix_status(B.DRAW_NORMAL, 0, 0, -1, out, 64) == B.ERR_INVALID_ARG
    assert B.draw_matrix_status(B.DRAW_NORMAL, 0, 0, 0, out, 65) == B.ERR_INVALID_ARG      # ld < d
    assert B.draw_matrix_status(B.DRAW_NORMAL, 0, 0, 0, out, 0) == B.ERR_INVALID_ARG
    assert B.lib().brace_draw_matrix(B.DRAW_NORMAL, 0, 0, 0, 2, 64, None, 64, 0.0, 1.0, None) == B.ERR_INVALID_ARG
    assert B.draw_matrix_status(B.DRAW_NORMAL, 0, 0, 0, out, 64) == B.OK
    torch.cuda.synchronize()


@pytest.mark.parametrize("name,d,ld", [("cfg2", 66_667, 66_688), ("cfg5", 80_000, 80_000), ("cfg2", 20_003, 20_005),
                                       ("cfg5", 20_003, 20_005)])
@pytest.mark.parametrize("ids", ["default", "scattered"])
def test_attacks_with_generated_draws(name, d, ld, ids):
    """Gaussian and sparse-noise attacks drawing inside the kernel: which coordinates are altered (the
    uniform test) is exact, the altered values are within tolerance, honest rows and padding stay."""
    w = W.scaled(W.WORKLOADS[name], d)
    seed, rnd = 2501017392 + w.n, 4
    H = W.honest_updates(w, 0, device="cuda", ld=ld)
    byz = list(range(w.f)) if ids == "default" else sorted(
        np.random.default_rng(w.n).choice(w.n, w.f, replace=False).tolist(), reverse=True)
    atk = B.make_attack(w.attack, sigma=w.sigma, prob=w.prob, byz_ids=None if ids == "default" else byz, seed=seed,
                        round_idx=rnd)
    ctx = B.Brace(w.n, w.f, w.d, B.default_params(lam=w.lam))
    U = H.clone()
    ctx.inject_attack(atk, H, U)
    U2 = H.clone()
    ctx.inject_attack(atk, U2, U2)
    assert torch.equal(U, U2)
    noise, unif = O.attack_draws(w.attack, seed, rnd, byz, d)
    exp = O.inject_attack(w.attack, H.cpu().numpy()[:, :d], byz, sigma=w.sigma, prob=w.prob, noise=noise, uniform=unif)
    got = U.cpu().numpy()
    honest = [i for i in range(w.n) if i not in byz]
    assert np.array_equal(got[honest, :d].view(np.uint32), exp[honest].view(np.uint32))
    assert_close_normals(got[byz, :d], exp[byz])
    if w.attack == B.ATTACK_SPARSE_NOISE:
        frac = float((got[byz, :d] != 0).mean())
        assert abs(frac - w.prob) < 0.01
    assert torch.equal(U[:, d:], H[:, d:])
    # the round on the library's own matrix against the oracle on the same bytes
    out = ctx.new_output()
    ctx.aggregate(U, out)
    bits = O.pack_bits_fast(O.gar_direct(got[:, :d], w.lam))
    res = out[:, : (d + 31) // 32].cpu().numpy().view(np.uint32)
    for c in range(w.n):
        assert np.array_equal(res[c], bits)
    ctx.close()


@pytest.mark.parametrize("d,ld", [(1_000_003, 1_000_064), (65_537, 65_539), (7, 8), (2048, 2048)])
@pytest.mark.parametrize("prob", [0.1, 0.0, 0.4999, 1e-4])
def test_sparse_noise_kernels_agree(d, ld, prob):
    """Attack 5 drawing in the kernel has two forms (normals computed for every block that needs one, or
    only for the compacted list of coordinate pairs that need one): same bits, at any prob and tail."""
    n, f = 5, 3
    H = torch.zeros((n, ld), dtype=torch.float32, device="cuda")
    rows = []
    for code in (0, 900):
        ctx = B.Brace(n, f, d)
        ctx.set_tuning(code, 0)
        U = torch.full_like(H, 3.0)
        ctx.inject_attack(B.make_attack(B.ATTACK_SPARSE_NOISE, sigma=2.5, prob=prob, byz_ids=[4, 0, 2], seed=31337,
                                        round_idx=9), H, U)
        rows.append(U)
        ctx.close()
    assert torch.equal(rows[0].view(torch.int32), rows[1].view(torch.int32))
    assert torch.equal(rows[0][[1, 3]], torch.full_like(H, 3.0)[[1, 3]])             # honest rows untouched
    assert (rows[0][:, d:] == 3.0).all()                                             # padding untouched
    frac = float((rows[0][[0, 2, 4], :d] != 0).float().mean())
    assert abs(frac - prob) < 0.02 + 3.0 / d ** 0.5
    if d <= 70_000:
        noise, unif = O.attack_draws(O.ATTACK_SPARSE_NOISE, 31337, 9, [4, 0, 2], d)
        exp = O.inject_attack(O.ATTACK_SPARSE_NOISE, np.zeros((n, d), np.float32), [4, 0, 2], sigma=2.5, prob=prob,
                              noise=noise, uniform=unif)
        assert_close_normals(rows[0].cpu().numpy()[[4, 0, 2], :d], exp[[4, 0, 2]])


def test_generated_draws_change_with_round_and_seed_and_bad_round_is_refused():
    w = W.scaled(W.WORKLOADS["cfg2"], 4_096)
    H = W.honest_updates(w, 0, device="cuda")
    ctx = B.Brace(w.n, w.f, w.d)
    rows = []
    for seed, rnd in ((1, 0), (1, 1), (2, 0)):
        U = H.clone()
        ctx.inject_attack(B.make_attack(w.attack, sigma=1.0, seed=seed, round_idx=rnd), H, U)
        rows.append(U[0].clone())
    assert not torch.equal(rows[0], rows[1]) and not torch.equal(rows[0], rows[2])
    bad = B.make_attack(w.attack, sigma=1.0, seed=1, round_idx=1 << 24)
    U = H.clone()
    assert B.lib().brace_inject_attack(ctx._ctx, bad, H.data_ptr(), H.stride(0), U.data_ptr(), U.stride(0),
                                       None) == B.ERR_INVALID_ARG
    bad2 = B.make_attack(w.attack, sigma=1.0)
    bad2.draws = 7
    assert B.lib().brace_inject_attack(ctx._ctx, bad2, H.data_ptr(), H.stride(0), U.data_ptr(), U.stride(0),
                                       None) == B.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert torch.equal(U, H)
    ctx.close()


def test_host_buffer_round_with_generated_draws():
    """brace_aggregate_host with the draws made on the device: only the updates cross the bus."""
    for name in ("cfg2", "cfg5"):
        w = W.scaled(W.WORKLOADS[name], 20_001)
        seed, rnd = 77, 2
        H = W.honest_updates(w, 0).pin_memory()
        atk = B.make_attack(w.attack, sigma=w.sigma, prob=w.prob, seed=seed, round_idx=rnd)
        ctx = B.Brace(w.n, w.f, w.d, B.default_params(lam=w.lam))
        d_out = ctx.new_output()
        h_out = torch.zeros(d_out.shape, dtype=d_out.dtype).pin_memory()
        d_U = torch.empty(H.shape, dtype=torch.float32, device="cuda")
        ctx.aggregate_host(atk, H, h_out, d_U, d_out)
        torch.cuda.synchronize()
        bits = O.pack_bits_fast(O.gar_direct(d_U.cpu().numpy()[:, :w.d], w.lam))
        got = h_out[:, : (w.d + 31) // 32].numpy().view(np.uint32)
        for c in range(w.n):
            assert np.array_equal(got[c], bits)
        noise, unif = O.attack_draws(w.attack, seed, rnd, list(range(w.f)), w.d)
        exp = O.inject_attack(w.attack, H.numpy()[:, :w.d], list(range(w.f)), sigma=w.sigma, prob=w.prob, noise=noise,
                              uniform=unif)
        assert_close_normals(d_U.cpu().numpy()[: w.f, :w.d], exp[: w.f])
        ctx.close()
