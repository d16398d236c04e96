"""Parity of the CUDA library against the CPU oracle, through the C ABI.

Integer work (signs, per-hop partial sign-sums, consensus bits, every client's
output row) must match bit for bit.  The plain-sum rule must match the oracle's
float32 ring-order sum bit for bit and the float64 sum within 1e-5 relative to
sum_i |g_i[k]| (the textbook forward-error scale of an n-term float32 sum)."""

import itertools

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


def dev(x: np.ndarray | torch.Tensor) -> torch.Tensor:
    t = torch.as_tensor(x)
    return t.cuda()


def expected_words(pm1_row: np.ndarray, d: int) -> np.ndarray:
    return O.pack_bits_fast(pm1_row, words=(d + 31) // 32)


def out_words(out: torch.Tensor, d: int) -> np.ndarray:
    """[n, ceil(d/32)] uint32 view of the library's output rows."""
    return out[:, : (d + 31) // 32].cpu().numpy().view(np.uint32)


def run_steps_and_check(ctx: B.Brace, U: torch.Tensor, tr: O.RingTrace, out: torch.Tensor, rule: int, d: int):
    """Drive the ring hop by hop; compare every client's mailbox after every hop."""
    n = ctx.n
    for s in range(n - 1):
        ctx.reduce_scatter_step(s, U)
        for r in range(n):
            seg, got = ctx.mailbox_tensor(r)
            exp_seg, exp = tr.rs_states[s][r]
            assert seg == exp_seg, (s, r)
            if rule == B.RULE_SUM:
                assert np.array_equal(got.numpy().view(np.uint32), exp.view(np.uint32)), (s, r)
            else:
                assert np.array_equal(got.numpy().astype(np.int32), exp), (s, r)
    ctx.consensus(out)
    for t in range(n - 1):
        ctx.allgather_step(t, out)
        if rule != B.RULE_SUM and tr.ag_states:
            # after hop t client r holds sub-vectors r+1, r, .., r-t (mod n) -- check the newest
            got = out_words(out, d)
            for r in range(n):
                j = (r - t) % n
                b, e = tr.bounds[j]
                bits = np.unpackbits(got[r].view(np.uint8), bitorder="little")[b:e]
                assert np.array_equal(bits, (tr.ag_states[t][r][b:e] > 0).astype(np.uint8)), (t, r)


def check_final(out: torch.Tensor, tr: O.RingTrace, rule: int, d: int):
    n = tr.outputs.shape[0]
    if rule == B.RULE_SUM:
        got = out[:, :d].cpu().numpy()
        for c in range(n):
            assert np.array_equal(got[c].view(np.uint32), tr.outputs[c].view(np.uint32)), c
    else:
        got = out_words(out, d)
        exp = expected_words(tr.outputs[0], d)
        for c in range(n):
            assert np.array_equal(got[c], exp), c


def final_mailboxes(ctx: B.Brace):
    return [[ctx.mailbox_tensor(c, hb) for c in range(ctx.n)] for hb in range(2 if ctx.n > 2 else 1)]


# ------------------------------------------------------------------ brute force on tiny inputs
@pytest.mark.parametrize("n", [2, 3, 4, 5])
def test_brute_force_all_sign_patterns(n):
    """All 3^n sign patterns at every coordinate, d = 1..8, lambda sweep, granules 1 / 2 / 128."""
    patterns = list(itertools.product([0, 1, 2], repeat=n))
    P = len(patterns)
    mags = np.array([0.5, 3.0, 1e-30, 7e20], dtype=np.float32)
    for d in range(1, 9):
        ld = 8
        out = torch.zeros((n, 4), dtype=torch.int32, device="cuda")
        for m in range(P):
            U = np.zeros((n, ld), dtype=np.float32)
            pats = [patterns[(m + k) % P] for k in range(d)]
            for k, pat in enumerate(pats):
                for i, t in enumerate(pat):
                    U[i, k] = (t - 1) * mags[(i + k) % 4]
            Ud = dev(U)
            settings = [(lam, 1) for lam in range(-n - 1, n + 1)] + [(lam, G) for G in (2, 128) for lam in (-1, 0, 1)]
            if m % 9:
                settings = [(0, 1), (1, 2), (-1, 128)]
            for lam, G in settings:
                tr = O.ring_round(U[:, :d], lam=lam, granule=G, keep_states=(m % 27 == 0))
                ctx = B.Brace(n, 0, d, B.default_params(lam=float(lam), granule=G))
                out.fill_(-1)
                if m % 27 == 0:
                    run_steps_and_check(ctx, Ud, tr, out, B.RULE_SIGN_CONSENSUS, d)
                    check_final(out, tr, B.RULE_SIGN_CONSENSUS, d)
                    out.fill_(-1)
                ctx.aggregate(Ud, out)
                check_final(out, tr, B.RULE_SIGN_CONSENSUS, d)
                ctx.close()


# ------------------------------------------------------------------ medium cases: several tiles + ragged tails
CASES = [
    # n, d, G, ld, lam, zero_sign
    (8, 100_000, 128, 100_096, 0.0, 0),
    (20, 70_001, 128, 70_004, 1.0, 0),
    (5, 4_099, 128, 4_100, 0.5, 1),
    (3, 1_000, 32, 1_000, 2.0, 0),
    (7, 12_345, 4, 12_348, -1.0, -1),
    (13, 50_001, 1, 50_001, 0.0, 0),
    (6, 33_000, 128, 33_024, 1.0, 0),
    (2, 5_000, 128, 5_000, 0.0, 0),
    (16, 300, 128, 384, 0.0, 0),          # fewer granules than clients: empty sub-vectors
    (9, 2_049, 128, 2_052, 3.0, 0),
]


@pytest.mark.parametrize("n,d,G,ld,lam,zs", CASES)
@pytest.mark.parametrize("rule", [B.RULE_SIGN_CONSENSUS, B.RULE_SUM])
def test_hop_by_hop_and_whole_round(n, d, G, ld, lam, zs, rule):
    U = W.small_integer_updates(n, d, seed=n + d, ld=ld) if (d % 2) else None
    if U is None:
        g = torch.Generator().manual_seed(n * 7 + d)
        U = torch.zeros((n, ld), dtype=torch.float32)
        U[:, :d].normal_(generator=g)
        U[:, :d][torch.rand((n, d), generator=g) < 0.15] = 0.0
    U[:, d:] = 123.0                                    # padding must never be read as data
    Uh = U.numpy()[:, :d]
    mean = 1 if (rule == B.RULE_SUM and n % 2) else 0
    tr = O.ring_round(Uh, rule=rule, lam=lam, zero_sign=zs, granule=G, mean=bool(mean))
    Ud = U.cuda()
    fusable = (G % 128 == 0) and (ld % 4 == 0)

    # (1) step calls, with per-hop parity
    ctx = B.Brace(n, 0, d, B.default_params(rule=rule, lam=lam, zero_sign=zs, granule=G, mean=mean,
                                            agg_mode=B.AGG_STEPWISE))
    out = ctx.new_output()
    out.fill_(-7 if rule != B.RULE_SUM else 0)
    run_steps_and_check(ctx, Ud, tr, out, rule, d)
    check_final(out, tr, rule, d)
    if rule == B.RULE_SIGN_CONSENSUS:
        assert np.array_equal(O.gar_direct(Uh, lam, zs), tr.outputs[0])
    boxes_steps = final_mailboxes(ctx)

    # (2) whole round, stepwise launches
    out2 = torch.full_like(out, 5)
    ctx.aggregate(Ud, out2)
    check_final(out2, tr, rule, d)
    for code in (10, 20, 40):                           # hop kernel with 1 / 2 / 4 float4 per thread
        ctx.set_tuning(code, 0)
        out2.fill_(5)
        ctx.aggregate(Ud, out2)
        check_final(out2, tr, rule, d)
        for c in range(n):
            assert torch.equal(ctx.mailbox_tensor(c)[1], boxes_steps[0][c][1])
    ctx.set_tuning(0, 0)

    # (3) whole round, fused kernel, every shape; mailboxes end as the step calls left them
    if fusable:
        # +1000 / +2000: share-only launch forced / never; a grid cap makes CTAs walk several tiles
        for variant, grid in [(v, 0) for v in range(0, 7)] + [(1001, 0), (2001, 0), (1006, 0), (2, 3), (6, 2)]:
            ctxf = B.Brace(n, 0, d, B.default_params(rule=rule, lam=lam, zero_sign=zs, granule=G, mean=mean,
                                                     agg_mode=B.AGG_FUSED))
            ctxf.workspace.fill_(0x5A)
            ctxf.set_tuning(variant, grid)
            out3 = torch.full_like(out, 9)
            ctxf.aggregate(Ud, out3)
            check_final(out3, tr, rule, d)
            boxes_fused = final_mailboxes(ctxf)
            for hb in range(len(boxes_steps)):
                for c in range(n):
                    seg_a, a = boxes_steps[hb][c]
                    seg_b, b2 = boxes_fused[hb][c]
                    assert seg_a == seg_b
                    assert torch.equal(a.view(torch.uint8), b2.view(torch.uint8)), (variant, hb, c)
            ctxf.close()
    else:
        ctxf = B.Brace(n, 0, d, B.default_params(rule=rule, lam=lam, zero_sign=zs, granule=G, agg_mode=B.AGG_FUSED))
        assert ctxf.aggregate_status(Ud, torch.zeros_like(out)) == B.ERR_UNSUPPORTED
        ctxf.close()
        ctxa = B.Brace(n, 0, d, B.default_params(rule=rule, lam=lam, zero_sign=zs, granule=G, mean=mean))
        out4 = torch.full_like(out, 3)
        ctxa.aggregate(Ud, out4)                        # AUTO falls back to stepwise launches
        check_final(out4, tr, rule, d)
        ctxa.close()

    # (4) plain sum against float64, relative to sum |g_i|
    if rule == B.RULE_SUM:
        ref = O.sum_direct_f64(Uh) / (n if mean else 1)
        scale = np.sum(np.abs(Uh.astype(np.float64)), axis=0) / (n if mean else 1)
        got = out2[0, :d].cpu().numpy().astype(np.float64)
        assert (np.abs(got - ref) <= REL_TOL * np.maximum(np.abs(ref), scale) + 1e-30).all()
    ctx.close()


@pytest.mark.parametrize("rule", [B.RULE_MAJORITY_SIGN, B.RULE_ABS_CONSENSUS])
@pytest.mark.parametrize("n,d,G,ld,lam", [(8, 100_000, 128, 100_096, 2.0), (5, 4_099, 128, 4_100, 1.5),
                                          (7, 12_345, 4, 12_348, 0.0), (20, 70_001, 128, 70_004, -1.0),
                                          (3, 1_000, 32, 1_000, 1.0), (128, 9_000, 128, 9_088, 30.0)])
def test_other_sign_rules(rule, n, d, G, ld, lam):
    """Majority sign and |S| > lambda on the same schedule: only the Phase III map differs."""
    U = W.small_integer_updates(n, d, seed=n * d, ld=ld, lo=-2, hi=2)
    Uh = U.numpy()[:, :d]
    tr = O.ring_round(Uh, rule=rule, lam=lam, granule=G)
    assert np.array_equal(tr.outputs[0], O.gar_direct(Uh, lam, rule=rule))
    Ud = U.cuda()
    ctx = B.Brace(n, 0, d, B.default_params(rule=rule, lam=lam, granule=G, agg_mode=B.AGG_STEPWISE))
    out = ctx.new_output()
    run_steps_and_check(ctx, Ud, tr, out, rule, d)
    check_final(out, tr, rule, d)
    ctx.close()
    ctxa = B.Brace(n, 0, d, B.default_params(rule=rule, lam=lam, granule=G))      # fused when the layout allows
    out2 = torch.full_like(out, 3)
    ctxa.aggregate(Ud, out2)
    check_final(out2, tr, rule, d)
    ctxa.close()


@pytest.mark.parametrize("rule,mean", [(B.RULE_SIGN_CONSENSUS, 0), (B.RULE_ABS_CONSENSUS, 0), (B.RULE_SUM, 0),
                                       (B.RULE_SUM, 1)])
@pytest.mark.parametrize("n,d,ldw", [(8, 100_001, 100_004), (5, 4_099, 4_101), (20, 33_000, 33_024)])
def test_model_update_after_round(rule, mean, n, d, ldw):
    """w <- w - eta * aggregate per client; float64 oracle, 1e-5 relative to the larger operand."""
    g = torch.Generator().manual_seed(n + d)
    U = torch.zeros((n, d + 3), dtype=torch.float32)
    U[:, :d].normal_(generator=g)
    Wt = torch.zeros((n, ldw), dtype=torch.float32)
    Wt.normal_(generator=g)
    eta = 0.03
    Uh, Wh = U.numpy()[:, :d], Wt.numpy().copy()
    tr = O.ring_round(Uh, rule=rule, lam=1.0, mean=bool(mean), keep_states=False)
    exp = O.apply_update(Wh[:, :d], tr.outputs, eta, rule, mean=bool(mean))
    ctx = B.Brace(n, 0, d, B.default_params(rule=rule, lam=1.0, mean=mean, agg_mode=B.AGG_STEPWISE))
    out = ctx.new_output()
    ctx.aggregate(U.cuda(), out)
    Wd = Wt.cuda()
    ctx.apply_update(out, Wd, eta)
    got = Wd.cpu().numpy()
    scale = np.maximum(np.abs(exp), np.abs(Wh[:, :d].astype(np.float64)))
    assert (np.abs(got[:, :d] - exp) <= REL_TOL * scale + 1e-30).all()
    assert np.array_equal(got[:, d:], Wh[:, d:])                       # row padding untouched
    if rule != B.RULE_SUM:                                             # one exact float32 subtraction of +-eta
        e32 = np.float32(eta)
        ref32 = Wh[:, :d] - e32 * tr.outputs.astype(np.float32)
        assert np.array_equal(got[:, :d].view(np.uint32), ref32.view(np.uint32))
    assert B.lib().brace_apply_update(ctx._ctx, out.data_ptr(), out.stride(0), Wd.data_ptr(), d - 1, eta,
                                      None) == B.ERR_INVALID_ARG   # rows shorter than d
    assert ctx.apply_update_status(out, Wd, float("nan")) == B.ERR_INVALID_ARG
    ctx.close()


@pytest.mark.parametrize("n", [2, 3, 4, 5, 8, 9, 16, 20, 33, 64, 65, 100, 128])
def test_coordinate_median_and_trimmed_mean(n):
    """The server-side coordinate-wise rules: sorted in registers, same bits as the oracle's
    sort + ascending float64 sum."""
    d, ld = 6_001, 6_003
    g = torch.Generator().manual_seed(n)
    U = torch.zeros((n, ld), dtype=torch.float32)
    U[:, :d].normal_(generator=g)
    U[:, :d][torch.rand((n, d), generator=g) < 0.1] = 0.0
    U[0, :50] = float("inf")
    U[n - 1, 25:75] = float("-inf")
    U[:, 100:110] = 3.25                                              # all clients equal
    U[:, d:] = float("nan")                                           # padding is never read
    Uh = U.numpy()[:, :d]
    ctx = B.Brace(n, 0, d, B.default_params(), host_only=True)        # needs no workspace
    Ud = U.cuda()
    res = torch.full((d + 8,), -7.0, dtype=torch.float32, device="cuda")
    ctx.coordinate_stat(B.STAT_MEDIAN, 0, Ud, res)
    got = res.cpu().numpy()
    exp = O.coordinate_median(Uh)
    assert np.array_equal(got[:d], exp, equal_nan=True)
    assert (got[d:] == -7.0).all()
    for trim in sorted({0, 1, n // 5, (n - 1) // 2}):
        if 2 * trim >= n:
            continue
        ctx.coordinate_stat(B.STAT_TRIMMED_MEAN, trim, Ud, res)
        got = res.cpu().numpy()[:d]
        exp = O.coordinate_trimmed_mean(Uh, trim)
        assert np.array_equal(got, exp, equal_nan=True), trim
    assert ctx.coordinate_stat_status(B.STAT_TRIMMED_MEAN, (n + 1) // 2, Ud, res) == B.ERR_INVALID_ARG
    assert ctx.coordinate_stat_status(B.STAT_TRIMMED_MEAN, -1, Ud, res) == B.ERR_INVALID_ARG
    assert ctx.coordinate_stat_status(7, 0, Ud, res) == B.ERR_INVALID_ARG
    ctx.close()
    if n == 128:
        big = B.Brace(129, 0, d, B.default_params(), host_only=True)
        assert big.coordinate_stat_status(B.STAT_MEDIAN, 0, Ud, res) == B.ERR_UNSUPPORTED
        big.close()


def test_unaligned_rows_fall_back_to_scalar_kernels():
    """Row stride not a multiple of 4 and a base pointer off 16 bytes."""
    n, d, ld = 6, 3_001, 3_003
    g = torch.Generator().manual_seed(5)
    buf = torch.zeros(n * ld + 1, dtype=torch.float32)
    buf.normal_(generator=g)
    Ud_full = buf.cuda()
    Ud = Ud_full[1:].view(n, ld)                        # 4-byte aligned only
    Uh = buf[1:].view(n, ld)[:, :d].numpy()
    for rule in (B.RULE_SIGN_CONSENSUS, B.RULE_SUM):
        tr = O.ring_round(Uh, rule=rule, lam=1.0, granule=128)
        ctx = B.Brace(n, 0, d, B.default_params(rule=rule, lam=1.0))
        out = ctx.new_output(out_ld=(d + 1) if rule == B.RULE_SUM else None)
        run_steps_and_check(ctx, Ud, tr, out, rule, d)
        check_final(out, tr, rule, d)
        out.zero_()
        ctx.aggregate(Ud, out)
        check_final(out, tr, rule, d)
        ctx.close()


def test_special_float_values():
    n, d = 9, 10_000
    U = W.edge_value_updates(n, d, seed=3, ld=10_112)
    Uh = U.numpy()[:, :d]
    for zs in (0, 1, -1):
        for lam in (0.0, -2.0, 2.5):
            tr = O.ring_round(Uh, lam=lam, zero_sign=zs, keep_states=False)
            ctx = B.Brace(n, 0, d, B.default_params(lam=lam, zero_sign=zs))
            out = ctx.new_output()
            ctx.aggregate(U.cuda(), out)
            check_final(out, tr, B.RULE_SIGN_CONSENSUS, d)
            ctx.close()
    # Phase I on its own
    ctx = B.Brace(n, 0, d)
    q = torch.zeros((n, d), dtype=torch.int8, device="cuda")
    ctx.quantize(U.cuda(), q)
    assert np.array_equal(q.cpu().numpy().astype(np.int32), O.sgn(Uh))
    ctx.close()


@pytest.mark.parametrize("n", [127, 128, 300])
def test_many_clients_partial_width(n):
    """int8 partial sums up to n = 127, int16 beyond; unanimous columns reach +-n."""
    d = 20_000
    g = torch.Generator().manual_seed(n)
    U = torch.zeros((n, d), dtype=torch.float32)
    U.normal_(generator=g)
    U[:, :64] = 1.0
    U[:, 64:128] = -1.0
    Uh = U.numpy()
    lam = float(n - 1)
    tr = O.ring_round(Uh, lam=lam, keep_states=False)
    assert tr.outputs[0][:64].tolist() == [1] * 64
    for mode in (B.AGG_STEPWISE, B.AGG_FUSED):
        ctx = B.Brace(n, 0, d, B.default_params(lam=lam, agg_mode=mode))
        out = ctx.new_output()
        ctx.aggregate(U.cuda(), out)
        check_final(out, tr, B.RULE_SIGN_CONSENSUS, d)
        j, owned = ctx.mailbox_tensor(n - 1)             # client n-1 owns sub-vector 0
        assert j == 0
        assert np.array_equal(owned.numpy().astype(np.int32), tr.owned[n - 1][1])
        ctx.close()


def test_largest_client_count():
    """n = 32767, the most the int16 partial sums hold: far more clients than granules, so
    most sub-vectors are empty; unanimous columns reach +-n without wrapping."""
    import ctypes
    n, d = 32767, 4096
    g = torch.Generator().manual_seed(7)
    U = torch.zeros((n, d), dtype=torch.float32)
    U.normal_(generator=g)
    U[:, :32] = 2.0
    U[:, 32:64] = -2.0
    Uh = U.numpy()
    S = O.sign_sum_direct(Uh)
    assert S[0] == n and S[32] == -n
    Ud = U.cuda()
    for rule, lam in ((B.RULE_SIGN_CONSENSUS, float(n - 1)), (B.RULE_SIGN_CONSENSUS, 100.0),
                      (B.RULE_ABS_CONSENSUS, float(n - 1))):
        exp = expected_words(O.gar_direct(Uh, lam, rule=rule), d)
        ctx = B.Brace(n, 0, d, B.default_params(rule=rule, lam=lam, agg_mode=B.AGG_FUSED))
        out = ctx.new_output()
        ctx.aggregate(Ud, out)
        assert (out_words(out, d) == exp[None, :]).all()
        ctx.close()
    # hop by hop: 65 533 launches; the owners' partials are the full sign-sums
    ctx = B.Brace(n, 0, d, B.default_params(lam=100.0, agg_mode=B.AGG_STEPWISE))
    out = ctx.new_output()
    ctx.aggregate(Ud, out)
    assert (out_words(out, d) == expected_words(O.gar_direct(Uh, 100.0), d)[None, :]).all()
    for j in (0, 1, 31):
        b, e = ctx.segment(j)
        if e > b:
            seg, box = ctx.mailbox_tensor((j - 1) % n)
            assert seg == j and np.array_equal(box.numpy().astype(np.int32), S[b:e])
    ctx.close()
    handle = ctypes.c_void_p()
    assert B.lib().brace_init(ctypes.byref(handle), n + 1, 0, d, B.default_params(), None, 0, None) == B.ERR_UNSUPPORTED


def test_rounds_are_memoryless():
    """Five consecutive rounds on one context equal five rounds on fresh contexts."""
    w = W.scaled(W.WORKLOADS["cfg5"], 40_000)
    ctx = B.Brace(w.n, w.f, w.d, B.default_params(lam=w.lam))
    out = ctx.new_output()
    for rnd in range(5):
        U = W.honest_updates(w, rnd, device="cuda")
        ctx.aggregate(U, out)
        fresh = B.Brace(w.n, w.f, w.d, B.default_params(lam=w.lam, agg_mode=B.AGG_STEPWISE))
        out_f = fresh.new_output()
        fresh.aggregate(U, out_f)
        assert torch.equal(out, out_f)
        tr = O.ring_round(U.cpu().numpy()[:, :w.d], lam=w.lam, keep_states=False)
        check_final(out, tr, B.RULE_SIGN_CONSENSUS, w.d)
        fresh.close()
    ctx.close()


def test_rounds_can_be_captured_in_a_cuda_graph():
    """Both round modes enqueue only kernels on the caller's stream, so a stream
    capture records them; replays on fresh inputs give the oracle's bits."""
    w = W.scaled(W.WORKLOADS["cfg2"], 70_001)
    U = W.honest_updates(w, 0, device="cuda")
    for mode in (B.AGG_FUSED, B.AGG_STEPWISE):
        ctx = B.Brace(w.n, w.f, w.d, B.default_params(lam=w.lam, agg_mode=mode))
        out = ctx.new_output()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            ctx.aggregate(U, out)
        torch.cuda.current_stream().wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            ctx.aggregate(U, out)
        for rnd in (1, 2):
            W.honest_updates(w, rnd, device="cuda", out=U)            # new data in the captured buffer
            out.fill_(-1)
            graph.replay()
            torch.cuda.synchronize()
            tr = O.ring_round(U.cpu().numpy()[:, :w.d], lam=w.lam, keep_states=False)
            check_final(out, tr, B.RULE_SIGN_CONSENSUS, w.d)
        del graph
        ctx.close()


def test_guard_bands_stay_untouched():
    """Canaries around the workspace, the output and the mailbox tails."""
    n, d, ld = 7, 9_001, 9_004
    g = torch.Generator().manual_seed(1)
    U = torch.zeros((n, ld), dtype=torch.float32)
    U[:, :d].normal_(generator=g)
    Ud = U.cuda()
    for rule in (B.RULE_SIGN_CONSENSUS, B.RULE_SUM):
        for mode in (B.AGG_STEPWISE, B.AGG_FUSED):
            p = B.default_params(rule=rule, agg_mode=mode)
            need = B.workspace_bytes(n, d, p)
            guard = 4096
            raw = torch.full((need + 2 * guard,), 0xA5, dtype=torch.uint8, device="cuda")
            ctx = B.Brace(n, 0, d, p, workspace=raw[guard: guard + need])
            words = (d + 31) // 32
            out_ld = (d + 4) if rule == B.RULE_SUM else words + 3
            if rule == B.RULE_SUM:
                out_ld = (out_ld + 3) // 4 * 4
            outbuf = torch.full((n + 2, out_ld), 0x3C3C3C3C, dtype=torch.int32, device="cuda")
            out = outbuf[1: n + 1]
            if rule == B.RULE_SUM:
                out = out.view(torch.float32)
            ctx.aggregate(Ud, out)
            torch.cuda.synchronize()
            assert (raw[:guard] == 0xA5).all() and (raw[guard + need:] == 0xA5).all()
            assert (outbuf[0] == 0x3C3C3C3C).all() and (outbuf[n + 1] == 0x3C3C3C3C).all()
            used = d if rule == B.RULE_SUM else words
            assert (outbuf[1: n + 1, used:] == 0x3C3C3C3C).all()
            tr = O.ring_round(U.numpy()[:, :d], rule=rule, keep_states=False)
            check_final(out, tr, rule, d)
            ctx.close()


# ------------------------------------------------------------------ API errors: status code, nothing launched
def test_step_order_and_argument_errors():
    n, d = 4, 1_000
    U = torch.zeros((n, d), dtype=torch.float32, device="cuda")
    ctx = B.Brace(n, 1, d)
    out = ctx.new_output()
    assert ctx.reduce_scatter_step_status(1, U) == B.ERR_BAD_STEP        # round not started
    assert ctx.consensus_status(out) == B.ERR_BAD_STEP
    assert ctx.allgather_step_status(0, out) == B.ERR_BAD_STEP
    assert ctx.reduce_scatter_step_status(0, U) == B.OK
    assert ctx.reduce_scatter_step_status(2, U) == B.ERR_BAD_STEP        # skipped hop 1
    assert ctx.reduce_scatter_step_status(n - 1, U) == B.ERR_BAD_STEP    # out of range
    assert ctx.reduce_scatter_step_status(-1, U) == B.ERR_BAD_STEP
    assert ctx.consensus_status(out) == B.ERR_BAD_STEP                   # reduce not finished
    assert ctx.reduce_scatter_step_status(1, U) == B.OK
    assert ctx.reduce_scatter_step_status(1, U) == B.ERR_BAD_STEP        # repeated hop
    assert ctx.reduce_scatter_step_status(2, U) == B.OK
    assert ctx.allgather_step_status(0, out) == B.ERR_BAD_STEP           # consensus first
    assert ctx.consensus_status(out) == B.OK
    assert ctx.consensus_status(out) == B.ERR_BAD_STEP
    assert ctx.allgather_step_status(1, out) == B.ERR_BAD_STEP
    for t in range(n - 1):
        assert ctx.allgather_step_status(t, out) == B.OK
    assert ctx.allgather_step_status(0, out) == B.ERR_BAD_STEP           # round is over
    assert ctx.reduce_scatter_step_status(0, U) == B.OK                  # step 0 restarts at any time
    assert ctx.reduce_scatter_step_status(0, U) == B.OK
    lib = B.lib()
    assert lib.brace_aggregate(ctx._ctx, None, d, out.data_ptr(), out.stride(0), None) == B.ERR_INVALID_ARG
    assert lib.brace_aggregate(ctx._ctx, U.data_ptr(), d - 1, out.data_ptr(), out.stride(0), None) == B.ERR_INVALID_ARG
    assert lib.brace_aggregate(ctx._ctx, U.data_ptr(), d, None, out.stride(0), None) == B.ERR_INVALID_ARG
    assert lib.brace_aggregate(ctx._ctx, U.data_ptr(), d, out.data_ptr(), (d + 31) // 32 - 1, None) == B.ERR_INVALID_ARG
    # attack argument checks
    a = B.make_attack(B.ATTACK_GAUSSIAN, sigma=1.0)                       # noise missing
    assert lib.brace_inject_attack(ctx._ctx, a, U.data_ptr(), d, U.data_ptr(), d, None) == B.ERR_INVALID_ARG
    a = B.make_attack(B.ATTACK_SCALE_OWN, byz_ids=[n])                    # id out of range
    assert lib.brace_inject_attack(ctx._ctx, a, U.data_ptr(), d, U.data_ptr(), d, None) == B.ERR_INVALID_ARG
    a = B.make_attack(9)
    assert lib.brace_inject_attack(ctx._ctx, a, U.data_ptr(), d, U.data_ptr(), d, None) == B.ERR_INVALID_ARG
    ctx2 = B.Brace(n, 2, d)
    a = B.make_attack(B.ATTACK_SCALE_OWN, byz_ids=[1, 1])                 # duplicate id
    assert lib.brace_inject_attack(ctx2._ctx, a, U.data_ptr(), d, U.data_ptr(), d, None) == B.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert ctx.last_cuda_error() == 0
    ctx.close()
    ctx2.close()


@pytest.mark.parametrize("n,d,zs", [(8, 700_001, 0), (3, 1_000_003, 1), (20, 1_663_370, 0), (50, 640_000, -1)])
def test_fused_round_medium_sizes(n, d, zs):
    """Launches of a few waves of CTAs (between the tiny parity cases and the full-size workloads): same
    bits as Eq. (1), same surviving mailboxes as the hop-by-hop round, several kernel shapes."""
    ld = W.round_up(d, 128)
    g = torch.Generator(device="cuda").manual_seed(n * 1000 + 7)
    U = torch.zeros((n, ld), dtype=torch.float32, device="cuda")
    U[:, :d].normal_(generator=g)
    U[:, :d][torch.rand((n, d), device="cuda", generator=g) < 0.05] = 0.0
    lam = float(n // 7)
    exp = O.pack_bits_fast(O.gar_direct(U.cpu().numpy()[:, :d], lam, zs))
    words = (d + 31) // 32
    ctx_s = B.Brace(n, 0, d, B.default_params(lam=lam, zero_sign=zs, agg_mode=B.AGG_STEPWISE))
    out_s = ctx_s.new_output()
    ctx_s.aggregate(U, out_s)
    boxes_s = final_mailboxes(ctx_s)
    for variant in (0, 6, 2, 1005):
        ctx = B.Brace(n, 0, d, B.default_params(lam=lam, zero_sign=zs, agg_mode=B.AGG_FUSED))
        ctx.workspace.fill_(0x33)
        ctx.set_tuning(variant, 0)
        out = torch.full_like(out_s, 5)
        ctx.aggregate(U, out)
        got = out[:, :words].cpu().numpy().view(np.uint32)
        for c in range(n):
            assert np.array_equal(got[c], exp), (variant, c)
        boxes = final_mailboxes(ctx)
        for hb in range(len(boxes_s)):
            for c in range(n):
                assert boxes[hb][c][0] == boxes_s[hb][c][0]
                assert torch.equal(boxes[hb][c][1], boxes_s[hb][c][1]), (variant, hb, c)
        ctx.close()
    ctx_s.close()


def test_random_shapes_rules_and_layouts():
    """Seeded random draws of (n, d, granule, row stride, rule, lambda, zero_sign, mean): the whole round by
    step calls with every mailbox compared after every hop, then by brace_aggregate in both modes, against
    the oracle's hop-by-hop trace.  Meant to hit combinations the hand-picked cases do not."""
    rng = np.random.default_rng(20250117392)
    rules = [B.RULE_SIGN_CONSENSUS, B.RULE_SUM, B.RULE_MAJORITY_SIGN, B.RULE_ABS_CONSENSUS]
    for case in range(40):
        n = int(rng.integers(2, 24))
        d = int(rng.choice([rng.integers(1, 40), rng.integers(40, 3000), rng.integers(3000, 40_000)]))
        G = int(rng.choice([1, 3, 4, 32, 100, 128, 256]))
        ld = d + int(rng.choice([0, 1, 2, 3, 4, 125]))
        if rng.random() < 0.5:
            ld = W.round_up(d, 128)
        rule = int(rng.choice(rules))
        lam = float(rng.integers(-n - 2, n + 2)) + float(rng.choice([0.0, 0.5]))
        zs = int(rng.choice([0, 0, 1, -1]))
        mean = int(rng.random() < 0.5)
        if rng.random() < 0.5:
            U = W.small_integer_updates(n, d, seed=case, ld=ld)
        else:
            U = W.edge_value_updates(n, d, seed=case, ld=ld)
            if rule == B.RULE_SUM:                     # NaN != NaN would hide nothing but complicates the compare
                U = torch.nan_to_num(U, nan=0.25, posinf=3.0, neginf=-3.0)
        Uh = U.numpy()[:, :d]
        with np.errstate(all="ignore"):
            tr = O.ring_round(Uh, rule=rule, lam=lam, zero_sign=zs, granule=G, mean=bool(mean))
        Ud = U.cuda()
        tag = (case, n, d, G, ld, rule, lam, zs, mean)
        ctx = B.Brace(n, 0, d, B.default_params(rule=rule, lam=lam, zero_sign=zs, granule=G, mean=mean,
                                                agg_mode=B.AGG_STEPWISE))
        out = ctx.new_output()
        run_steps_and_check(ctx, Ud, tr, out, rule, d)
        check_final(out, tr, rule, d)
        out.fill_(0)
        ctx.aggregate(Ud, out)
        check_final(out, tr, rule, d)
        ctx.close()
        ctxa = B.Brace(n, 0, d, B.default_params(rule=rule, lam=lam, zero_sign=zs, granule=G, mean=mean,
                                                 agg_mode=B.AGG_AUTO))
        outa = ctxa.new_output()
        ctxa.aggregate(Ud, outa)
        try:
            check_final(outa, tr, rule, d)
        except AssertionError as exc:
            raise AssertionError(f"case {tag}: {exc}") from exc
        ctxa.close()


def test_inject_inside_stream_capture():
    """The Byzantine id list is uploaded by the first call that sees it.  That upload must not be recorded
    into a graph (later eager calls would skip it): a capturing call with a new list is refused, and after
    one eager call the same list captures and replays fine."""
    w = W.scaled(W.WORKLOADS["cfg3"], 20_000)
    H = W.honest_updates(w, 0, device="cuda")
    byz = [7, 3, 41, 20, 11, 0, 49, 30, 5, 17]
    atk = B.make_attack(w.attack, scale=w.scale, byz_ids=byz)
    ctx = B.Brace(w.n, w.f, w.d, B.default_params(lam=w.lam))
    U, out = H.clone(), ctx.new_output()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        status = B.lib().brace_inject_attack(ctx._ctx, atk, H.data_ptr(), H.stride(0), U.data_ptr(), U.stride(0),
                                             torch.cuda.current_stream().cuda_stream)
        out.fill_(0)                                     # the graph must not be empty
    assert status == B.ERR_UNSUPPORTED
    assert torch.equal(U, H)
    ctx.inject_attack(atk, H, U)                         # eager: uploads the list
    ctx.aggregate(U, out)
    torch.cuda.synchronize()
    exp_u, exp_out = U.clone(), out.clone()
    exp = O.inject_attack(w.attack, H.cpu().numpy()[:, :w.d], byz, scale=w.scale)
    assert np.array_equal(exp_u.cpu().numpy()[:, :w.d].view(np.uint32), exp.view(np.uint32))
    U.copy_(H)
    out.fill_(0)
    graph2 = torch.cuda.CUDAGraph()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(graph2, stream=side):
        ctx.inject_attack(atk, H, U)
        ctx.aggregate(U, out)
    U.copy_(H)
    out.fill_(0)
    graph2.replay()
    torch.cuda.synchronize()
    assert torch.equal(U, exp_u) and torch.equal(out, exp_out)
    ctx.close()


# ------------------------------------------------------------------ attack injection + whole pipeline
def _np(t):
    return None if t is None else t.cpu().numpy()


@pytest.mark.parametrize("name,d", [("cfg1", 100_000), ("cfg2", 66_667), ("cfg3", 50_002), ("cfg4", 30_001),
                                    ("cfg5", 80_000)])
@pytest.mark.parametrize("ids", ["default", "scattered"])
def test_attack_injection_and_pipeline(name, d, ids):
    w = W.scaled(W.WORKLOADS[name], d)
    H = W.honest_updates(w, 0, device="cuda")
    noise, unif = W.attack_draws(w, 0, device="cuda")
    byz = list(range(w.f)) if ids == "default" else sorted(
        np.random.default_rng(w.n).choice(w.n, w.f, replace=False).tolist(), reverse=True)
    atk = B.make_attack(w.attack, scale=w.scale, sigma=w.sigma, kappa=w.kappa, prob=w.prob,
                        byz_ids=None if ids == "default" else byz, noise=noise, uniform=unif)
    ctx = B.Brace(w.n, w.f, w.d, B.default_params(lam=w.lam))
    U = H.clone()
    ctx.inject_attack(atk, H, U)                                           # separate source and destination
    U2 = H.clone()
    ctx.inject_attack(atk, U2, U2)                                         # in place
    assert torch.equal(U, U2)
    Hh = H.cpu().numpy()[:, :d]
    exp = O.inject_attack(w.attack, Hh, byz, scale=w.scale, sigma=w.sigma, kappa=w.kappa, prob=w.prob,
                          noise=None if noise is None else _np(noise)[:, :d],
                          uniform=None if unif is None else _np(unif)[:, :d])
    got = U.cpu().numpy()[:, :d]
    denom = np.maximum(np.abs(exp), 1e-30)
    assert (np.abs(got - exp) / denom).max() <= REL_TOL
    assert np.array_equal(np.sign(got), np.sign(exp))                      # the votes are identical
    assert np.array_equal(got.view(np.uint32), exp.view(np.uint32))        # and, by construction, the bits
    assert torch.equal(U[:, d:], H[:, d:])                                 # padding untouched
    # ring on the library's own injected matrix vs oracle on the oracle's
    out = ctx.new_output()
    ctx.aggregate(U, out)
    tr = O.ring_round(exp, lam=w.lam, keep_states=False)
    check_final(out, tr, B.RULE_SIGN_CONSENSUS, d)
    assert np.array_equal(tr.outputs[0], O.gar_direct(exp, w.lam))
    ctx.close()


@pytest.mark.parametrize("n,f", [(100, 20), (9, 2), (37, 5), (128, 1), (12, 11)])
def test_mean_shift_statistics_special_values(n, f):
    """Honest rows sprinkled with +-0, denormals, +-FLT_MAX, +-Inf and NaN: the statistics kernel widens
    float32 to float64 with integer operations where every input of a coordinate is a normal number and
    falls back to the conversion instruction elsewhere; both routes must give the oracle's bits (a
    coordinate whose oracle value is NaN must be NaN)."""
    d, ld = 6_000, 6_016
    H = W.edge_value_updates(n, d, seed=n, ld=ld)
    Hn = H.numpy()
    Hn[:, : d // 2] = np.where(np.isfinite(Hn[:, : d // 2]), Hn[:, : d // 2], np.float32(0.25))   # first half: no Inf / NaN
    Hn[:, : d // 4] = np.where(np.abs(Hn[:, : d // 4]) > 1e30, np.float32(-3.0), Hn[:, : d // 4])  # first quarter: no overflow
    g = torch.Generator().manual_seed(7 * n)
    Hn[:, 100:1100] = torch.empty((n, 1000)).normal_(0.0, 0.01, generator=g).numpy()               # all-normal columns
    for kind, kw in ((B.ATTACK_MEAN_SHIFT, dict(kappa=3.0)), (B.ATTACK_SCALED_MEAN, dict(scale=-5.0))):
        ctx = B.Brace(n, f, d)
        U = H.cuda()
        ctx.inject_attack(B.make_attack(kind, **kw), U, U)
        with np.errstate(all="ignore"):
            exp = O.inject_attack(kind, Hn[:, :d], list(range(f)), **kw)
        got = U.cpu().numpy()[:, :d]
        nan = np.isnan(exp)
        assert np.array_equal(np.isnan(got), nan)
        assert nan[:, : d // 2].sum() == 0 and nan.sum() > 0
        assert np.array_equal(got.view(np.uint32)[~nan], exp.view(np.uint32)[~nan])
        ctx.close()


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
def test_attack_injection_unaligned_rows(name):
    """Row strides that are not multiples of 4 take the scalar kernels; same bits."""
    d, ld = 20_003, 20_005
    w = W.scaled(W.WORKLOADS[name], d)
    H = W.honest_updates(w, 1, device="cuda", ld=ld)
    noise, unif = W.attack_draws(w, 1, device="cuda", ld=ld + 2)
    atk = B.make_attack(w.attack, scale=w.scale, sigma=w.sigma, kappa=w.kappa, prob=w.prob, noise=noise, uniform=unif)
    ctx = B.Brace(w.n, w.f, w.d, B.default_params(lam=w.lam))
    U = H.clone()
    ctx.inject_attack(atk, H, U)
    exp = O.inject_attack(w.attack, H.cpu().numpy()[:, :d], list(range(w.f)), scale=w.scale, sigma=w.sigma,
                          kappa=w.kappa, prob=w.prob, noise=None if noise is None else _np(noise)[:, :d],
                          uniform=None if unif is None else _np(unif)[:, :d])
    got = U.cpu().numpy()
    assert np.array_equal(got[:, :d].view(np.uint32), exp.view(np.uint32))
    assert torch.equal(U[:, d:], H[:, d:])
    ctx.close()


def test_host_buffer_round():
    """brace_aggregate_host: pinned host in, host out, attack applied on the device copy."""
    for name in ("cfg2", "cfg5", "cfg4"):
        w = W.scaled(W.WORKLOADS[name], 20_001)
        H = W.honest_updates(w, 0).pin_memory()
        noise, unif = W.attack_draws(w, 0)
        atk = B.make_attack(w.attack, scale=w.scale, sigma=w.sigma, kappa=w.kappa, prob=w.prob,
                            noise=None if noise is None else noise.pin_memory(),
                            uniform=None if unif is None else unif.pin_memory())
        ctx = B.Brace(w.n, w.f, w.d, B.default_params(lam=w.lam))
        d_out = ctx.new_output()
        h_out = torch.zeros(d_out.shape, dtype=d_out.dtype).pin_memory()
        d_U = torch.empty(H.shape, dtype=torch.float32, device="cuda")
        d_noise = None if noise is None else torch.empty(noise.shape, dtype=torch.float32, device="cuda")
        d_unif = None if unif is None else torch.empty(unif.shape, dtype=torch.float32, device="cuda")
        ctx.aggregate_host(atk, H, h_out, d_U, d_out, d_noise, d_unif)
        torch.cuda.synchronize()
        exp = O.inject_attack(w.attack, H.numpy()[:, :w.d], list(range(w.f)), scale=w.scale, sigma=w.sigma,
                              kappa=w.kappa, prob=w.prob, noise=None if noise is None else noise.numpy()[:, :w.d],
                              uniform=None if unif is None else unif.numpy()[:, :w.d])
        tr = O.ring_round(exp, lam=w.lam, keep_states=False)
        got = h_out[:, : (w.d + 31) // 32].numpy().view(np.uint32)
        ew = expected_words(tr.outputs[0], w.d)
        for c in range(w.n):
            assert np.array_equal(got[c], ew)
        ctx.close()
