"""Parity at the full sizes of the five workloads, in the launch configuration
bench.py times (fused round, default tuning; injection in its default kernels,
attacks 2 and 5 drawing inside the kernel).

Every bit is compared: the device matrices are streamed back in coordinate
slabs, the oracle runs on each slab (Eq. (1) is per coordinate, so a slab is an
independent problem) and is compared with every output word of client 0's row
and with every owner's final sign-sums; the other clients' rows are compared
with client 0's on the device.  A sampled comparison runs first as a fast
pre-check.  Slabs are handed to a few host threads (numpy releases the GIL);
each thread calls the oracle as it stands."""

import concurrent.futures as cf
import os

import numpy as np
import pytest
import torch

from oracle import brace_oracle as O
from paper_2501_17392_b200 import brace as B
from paper_2501_17392_b200 import build as brace_build
from paper_2501_17392_b200 import workloads as W

pytestmark = pytest.mark.gpu
REL_TOL = 1e-5
THREADS = max(1, min(12, len(os.sched_getaffinity(0))))


@pytest.fixture(scope="module", autouse=True)
def _built():
    brace_build.build()
    assert torch.cuda.is_available(), "these tests need a CUDA device"


def sample_coordinates(ctx: B.Brace, d: int, n: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng(seed)
    picks = [np.arange(0, min(d, 2048)), np.arange(max(0, d - 2048), d), rng.integers(0, d, size=8192)]
    for j in sorted(set([0, 1, n // 2, n - 2, n - 1])):
        b, e = ctx.segment(j)
        picks.append(np.arange(max(0, b - 64), min(d, b + 64)))
        picks.append(np.arange(max(0, e - 64), min(d, e + 64)))
    return np.unique(np.concatenate(picks)).astype(np.int64)


def bits_at(row_words: torch.Tensor, idx: torch.Tensor) -> np.ndarray:
    w = row_words[idx // 32].to(torch.int64) & 0xFFFFFFFF
    return ((w >> (idx % 32)) & 1).cpu().numpy().astype(np.int8)


def slab_width(n: int) -> int:
    """Coordinates per slab: a multiple of 128, about 2e8 elements per slab at most."""
    return int(max(1 << 18, min(1 << 22, (200_000_000 // n) // 128 * 128)))


def owners_sign_sums(ctx: B.Brace, n: int) -> torch.Tensor:
    """The d final sign-sums, gathered from the mailboxes of the sub-vectors' owners
    (client j-1 owns sub-vector j) in coordinate order, on the device."""
    parts = []
    for j in range(n):
        owner = (j - 1) % n
        p, ln, seg, eb = ctx.debug_mailbox(owner, 0)
        assert seg == j and eb == 1
        off = p - ctx.workspace.data_ptr()
        parts.append(ctx.workspace[off: off + ln].view(torch.int8))
    return torch.cat(parts)


def check_slab(w, lam, byz, U_slab, out_words, sums, start, atk_check):
    """Oracle on one slab of all n rows against the result words and sign-sums of the same coordinates."""
    width = U_slab.shape[1]
    total = O.sign_sum_direct(U_slab)
    assert np.array_equal(total.astype(np.int8), sums), f"sign-sums differ in slab at {start}"
    pm1 = O.consensus_map(total, O.RULE_SIGN_CONSENSUS, lam, w.n)
    exp_words = O.pack_bits_fast(pm1)
    assert np.array_equal(exp_words, out_words), f"output words differ in slab at {start}"
    if start == 0:                                    # the definition in one piece, once
        assert np.array_equal(O.gar_direct(U_slab[:, :65536], lam), pm1[:65536])
    if atk_check is None or not byz:
        return
    if w.attack in (O.ATTACK_SCALED_MEAN, O.ATTACK_MEAN_SHIFT):
        # the honest rows of the injected matrix are the honest matrix (checked on the device)
        exp = O.inject_attack(w.attack, U_slab, byz, scale=w.scale, kappa=w.kappa)
        assert np.array_equal(exp[byz].view(np.uint32), U_slab[byz].view(np.uint32)), f"injected rows differ at {start}"
    elif w.attack in (O.ATTACK_GAUSSIAN, O.ATTACK_SPARSE_NOISE):
        seed, rnd = atk_check
        noise, unif = O.attack_draws(w.attack, seed, rnd, byz, width, start=start)
        exp = O.inject_attack(w.attack, U_slab, byz, sigma=w.sigma, prob=w.prob, noise=noise, uniform=unif)[byz]
        got = U_slab[byz]
        assert np.array_equal(got == 0, exp == 0), f"altered coordinates differ at {start}"
        assert (np.abs(got.astype(np.float64) - exp) <= REL_TOL * np.abs(exp.astype(np.float64))).all()


def full_compare(w, ctx, U, out, lam, byz, atk_check, draws_every=1):
    """Every output word of row 0 and every final sign-sum against the oracle, slab by slab; rows 1..n-1
    against row 0 on the device."""
    n, d = w.n, w.d
    words = (d + 31) // 32
    for c in range(1, n):
        assert torch.equal(out[c, :words], out[0, :words]), f"client {c} differs from client 0"
    if d % 32:
        assert (int(out[0, words - 1].item()) & 0xFFFFFFFF) >> (d % 32) == 0, "padding bits must be zero"
    sums_dev = owners_sign_sums(ctx, n)
    assert sums_dev.numel() == d
    out0 = out[0, :words].cpu().numpy().view(np.uint32)
    sums = sums_dev.cpu().numpy()
    del sums_dev
    S = slab_width(n)
    starts = list(range(0, d, S))
    stats_attack = w.attack in (O.ATTACK_SCALED_MEAN, O.ATTACK_MEAN_SHIFT)
    with cf.ThreadPoolExecutor(max_workers=THREADS) as pool:
        pending = []
        for i, a in enumerate(starts):
            b = min(d, a + S)
            U_slab = U[:, a:b].cpu().numpy()
            check = atk_check if (stats_attack or i % draws_every == 0 or i == len(starts) - 1) else None
            pending.append(pool.submit(check_slab, w, lam, byz, U_slab, out0[a // 32: (b + 31) // 32], sums[a:b], a,
                                       check))
            while len(pending) > THREADS + 2:
                pending.pop(0).result()
        for fut in pending:
            fut.result()


def sampled_precheck(w, ctx, U, out, lam):
    idx_np = sample_coordinates(ctx, w.d, w.n, seed=w.n)
    idx = torch.as_tensor(idx_np, device="cuda")
    cols = U[:, idx].cpu().numpy()
    assert np.array_equal(bits_at(out[0], idx), (O.gar_direct(cols, lam) > 0).astype(np.int8))


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4", "cfg5"])
def test_full_size_workload(name):
    w = W.WORKLOADS[name]
    n, f, d = w.n, w.f, w.d
    ctx = B.Brace(n, f, d, B.default_params(lam=w.lam, agg_mode=B.AGG_FUSED))
    H = torch.zeros((n, w.ld), dtype=torch.float32, device="cuda")
    U = torch.empty_like(H)
    out = ctx.new_output()
    byz = list(range(f))
    generated = w.attack in (W.ATTACK_GAUSSIAN, W.ATTACK_SPARSE_NOISE)
    seed = W.BASE_SEED + n
    for rnd in range(w.rounds):
        W.honest_updates(w, rnd, device="cuda", out=H)
        U.copy_(H)
        atk = B.make_attack(w.attack, scale=w.scale, sigma=w.sigma, kappa=w.kappa, prob=w.prob,
                            seed=seed if generated else None, round_idx=rnd)
        ctx.inject_attack(atk, H, U)
        assert torch.equal(U[f:], H[f:]), "honest rows must not change"
        assert torch.equal(U[:, d:], H[:, d:]), "row padding must not change"
        out.fill_(-1)
        ctx.aggregate(U, out)
        torch.cuda.synchronize()
        sampled_precheck(w, ctx, U, out, w.lam)
        full_compare(w, ctx, U, out, w.lam, byz, (seed, rnd), draws_every=4 if name == "cfg5" else 1)
    # the hop-by-hop path on the same (last) inputs: same bits, same surviving mailboxes
    del H
    torch.cuda.empty_cache()
    ctx_s = B.Brace(n, f, d, B.default_params(lam=w.lam, agg_mode=B.AGG_STEPWISE))
    out_s = ctx_s.new_output()
    ctx_s.aggregate(U, out_s)
    torch.cuda.synchronize()
    words = (d + 31) // 32
    assert torch.equal(out_s[:, :words], out[:, :words])
    for c in range(n):
        for hb in (0, 1):
            pa, la, sa, _ = ctx.debug_mailbox(c, hb)
            pb, lb, sb, _ = ctx_s.debug_mailbox(c, hb)
            assert sa == sb and la == lb
            oa, ob = pa - ctx.workspace.data_ptr(), pb - ctx_s.workspace.data_ptr()
            assert torch.equal(ctx.workspace[oa: oa + la], ctx_s.workspace[ob: ob + lb])
    ctx.close()
    ctx_s.close()
    del U, out, out_s
    torch.cuda.empty_cache()


def test_full_size_cfg1_with_its_attack():
    """cfg1 at its real size (small enough for the oracle's hop-by-hop procedure in full)."""
    w = W.WORKLOADS["cfg1"]
    H = W.honest_updates(w, 0, device="cuda")
    U = H.clone()
    ctx = B.Brace(w.n, w.f, w.d, B.default_params(lam=w.lam, agg_mode=B.AGG_FUSED))
    ctx.inject_attack(B.make_attack(w.attack, scale=w.scale), H, U)
    out = ctx.new_output()
    ctx.aggregate(U, out)
    torch.cuda.synchronize()
    exp_u = O.inject_attack(w.attack, H.cpu().numpy()[:, :w.d], list(range(w.f)), scale=w.scale)
    assert np.array_equal(U.cpu().numpy()[:, :w.d].view(np.uint32), exp_u.view(np.uint32))
    tr = O.ring_round(exp_u, lam=w.lam, keep_states=False)
    words = (w.d + 31) // 32
    got = out[:, :words].cpu().numpy().view(np.uint32)
    for c in range(w.n):
        assert np.array_equal(got[c], O.pack_bits_fast(tr.outputs[c]))
    full_compare(w, ctx, U, out, w.lam, list(range(w.f)), None)
    ctx.close()


def test_vector_longer_than_2_to_31():
    """Two clients, d just above 2^31: every in-row offset needs 64-bit arithmetic.  Every output
    word against Eq. (1), both round modes, plus the attack and model-update kernels at the far end of
    the rows."""
    n, d = 2, (1 << 31) + 4_099
    ld = W.round_up(d, 128)
    free, _ = torch.cuda.mem_get_info()
    if free < 3 * n * ld * 4:
        pytest.skip("not enough free device memory for a 2 x 2^31 float32 matrix")
    U = torch.empty((n, ld), dtype=torch.float32, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(99)
    for i in range(n):
        U[i].normal_(generator=g)
    U[:, d:].zero_()
    w = W.Workload("long", n, 1, d, 1, "gauss", W.ATTACK_SCALE_OWN, scale=-10.0)
    ctx = B.Brace(n, 1, d, B.default_params(lam=0.0, agg_mode=B.AGG_FUSED))
    rng = np.random.default_rng(5)
    b1, e1 = ctx.segment(1)
    picks = [np.arange(0, 1024), np.arange((1 << 31) - 600, (1 << 31) + 600), np.arange(b1 - 300, b1 + 300),
             np.arange(d - 1500, d), rng.integers(0, d, 4096)]
    idx_np = np.unique(np.concatenate(picks)).astype(np.int64)
    idx = torch.as_tensor(idx_np, device="cuda")
    # attack 1 on client 0 (own update scaled), then the round
    atk = B.make_attack(B.ATTACK_SCALE_OWN, scale=-10.0)
    Hs = U[:, idx].cpu().numpy()
    ctx.inject_attack(atk, U, U)
    Us = U[:, idx].cpu().numpy()
    exp_u = O.inject_attack(O.ATTACK_SCALE_OWN, Hs, [0], scale=-10.0)
    assert np.array_equal(Us.view(np.uint32), exp_u.view(np.uint32))
    out = ctx.new_output()
    ctx.aggregate(U, out)
    torch.cuda.synchronize()
    words = (d + 31) // 32
    exp_bits = (O.gar_direct(exp_u, 0.0) > 0).astype(np.int8)
    assert np.array_equal(bits_at(out[0], idx), exp_bits)
    full_compare(w, ctx, U, out, 0.0, [0], None)
    ctx_s = B.Brace(n, 1, d, B.default_params(lam=0.0, agg_mode=B.AGG_STEPWISE))
    out_s = ctx_s.new_output()
    ctx_s.aggregate(U, out_s)
    torch.cuda.synchronize()
    assert torch.equal(out_s[:, :words], out[:, :words])
    # model update in place on the update matrix itself (used here as the parameter rows)
    before = U[:, idx].cpu().numpy()
    ctx.apply_update(out, U, 0.5)
    after = U[:, idx].cpu().numpy()
    sign = np.where(exp_bits > 0, 1.0, -1.0).astype(np.float32)
    assert np.array_equal(after, before - np.float32(0.5) * sign[None, :])
    ctx.close()
    ctx_s.close()
    del U, out, out_s
    torch.cuda.empty_cache()


def test_full_size_sum_rule_cfg2():
    """Plain ring-all-reduce at cfg2's size: fused and hop-by-hop give the same float32 bits, and every
    coordinate matches the float32 ring-order sum (sub-vector j is reduced starting at client j) and the
    oracle's float64 sum within tolerance."""
    w = W.WORKLOADS["cfg2"]
    H = W.honest_updates(w, 0, device="cuda")
    outs = []
    for mode, tuning in ((B.AGG_FUSED, 0), (B.AGG_STEPWISE, 0), (B.AGG_FUSED, 1000)):   # 1000: owner rows + share-only launch
        ctx = B.Brace(w.n, 0, w.d, B.default_params(rule=B.RULE_SUM, agg_mode=mode))
        ctx.set_tuning(tuning, 0)
        out = ctx.new_output()
        ctx.aggregate(H, out)
        torch.cuda.synchronize()
        outs.append(out)
        bounds = [ctx.segment(j) for j in range(w.n)]
        ctx.close()
    assert torch.equal(outs[0][:, :w.d].view(torch.int32), outs[1][:, :w.d].view(torch.int32))
    assert torch.equal(outs[0][:, :w.d].view(torch.int32), outs[2][:, :w.d].view(torch.int32))
    for c in range(1, w.n):
        assert torch.equal(outs[0][c, :w.d].view(torch.int32), outs[0][0, :w.d].view(torch.int32))
    Hh = H.cpu().numpy()[:, :w.d]
    got = outs[0][0, :w.d].cpu().numpy()
    for j, (b, e) in enumerate(bounds):
        acc = Hh[j, b:e].copy()
        for i in range(1, w.n):
            acc = (acc + Hh[(j + i) % w.n, b:e]).astype(np.float32)     # float32 adds, ring order
        assert np.array_equal(got[b:e].view(np.uint32), acc.view(np.uint32)), f"sub-vector {j}"
    ref = O.sum_direct_f64(Hh)
    scale = np.abs(Hh.astype(np.float64)).sum(0)
    assert (np.abs(got.astype(np.float64) - ref) <= 1e-5 * np.maximum(np.abs(ref), scale)).all()
