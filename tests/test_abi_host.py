"""The C-ABI library loads on a machine without a GPU, exports every function
include/brace.h declares, and its host-side logic (argument checks, partition,
workspace size, step-order validation entry conditions) behaves as documented.
No kernel is launched here."""

import ctypes as C
import os
import re

import pytest

from oracle import brace_oracle as O
from paper_2501_17392_b200 import brace as B
from paper_2501_17392_b200 import build as brace_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    brace_build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "brace.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(brace_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = _declared()
    assert "brace_init" in names and "brace_aggregate" in names and len(names) >= 15
    handle = C.CDLL(B.LIB_PATH)
    for name in names:
        assert hasattr(handle, name), name
        assert name in B.SIGNATURES, f"{name} has no binding"
    assert sorted(B.SIGNATURES) == names


def test_status_strings_and_defaults():
    assert B.status_string(B.OK) == "ok"
    for s in range(1, 7):
        assert B.status_string(s) and B.status_string(s) != "ok"
    p = B.default_params()
    assert (p.rule, p.lam, p.zero_sign, p.granule, p.mean, p.agg_mode) == (0, 0.0, 0, 128, 0, 0)
    assert B.lib().brace_default_params(None) == B.ERR_INVALID_ARG


@pytest.mark.parametrize("n,d,G", [(3, 3, 1), (4, 10, 1), (5, 3, 1), (8, 100000, 128), (20, 1663370, 128),
                                   (50, 11689512, 128), (100, 25557032, 128), (16, 124439808, 128), (5, 8, 2),
                                   (5, 8, 128), (7, 1000, 32), (127, 5000, 4), (300, 70000, 128), (2, 1, 1)])
def test_partition_matches_oracle(n, d, G):
    ctx = B.Brace(n, 0, d, B.default_params(granule=G), host_only=True)
    assert [ctx.segment(j) for j in range(n)] == O.partition(n, d, G)
    with pytest.raises(B.BraceError):
        ctx.segment(n)
    with pytest.raises(B.BraceError):
        ctx.segment(-1)
    ctx.close()


def test_init_argument_errors():
    lib = B.lib()
    p = B.default_params()
    ctx = C.c_void_p()

    def init(n, f, d, params=p, ws=None, nbytes=0):
        return lib.brace_init(C.byref(ctx), n, f, d, C.byref(params) if params is not None else None, ws, nbytes, None)

    assert init(1, 0, 10) == B.ERR_INVALID_ARG
    assert init(4, 4, 10) == B.ERR_INVALID_ARG
    assert init(4, -1, 10) == B.ERR_INVALID_ARG
    assert init(4, 1, 0) == B.ERR_INVALID_ARG
    assert init(4, 1, 10, params=None) == B.ERR_INVALID_ARG
    assert lib.brace_init(None, 4, 1, 10, C.byref(p), None, 0, None) == B.ERR_INVALID_ARG
    for bad in [dict(rule=7), dict(lam=float("nan")), dict(lam=float("inf")), dict(zero_sign=2), dict(granule=0),
                dict(agg_mode=9)]:
        assert init(4, 1, 10, params=B.default_params(**bad)) == B.ERR_INVALID_ARG, bad
    assert init(40000, 1, 10) == B.ERR_UNSUPPORTED
    assert init(40000, 1, 10, params=B.default_params(rule=B.RULE_SUM)) == B.OK   # float mailboxes: no width limit
    lib.brace_destroy(ctx)
    # a workspace that is too small or misaligned is refused (the pointer is never dereferenced)
    need = B.workspace_bytes(4, 1000, p)
    assert need > 0
    assert init(4, 1, 1000, ws=4096, nbytes=need - 1) == B.ERR_WORKSPACE
    assert init(4, 1, 1000, ws=4096 + 8, nbytes=need) == B.ERR_WORKSPACE
    assert init(4, 1, 1000, ws=None, nbytes=need) == B.ERR_WORKSPACE
    assert lib.brace_destroy(None) == B.ERR_INVALID_ARG


def test_workspace_bytes():
    p = B.default_params()
    assert B.workspace_bytes(1, 10, p) == 0
    assert B.workspace_bytes(4, 0, p) == 0
    # two mailbox sets of n * padded longest sub-vector, plus the id lists
    n, d = 8, 100000
    longest = max(e - b for b, e in O.partition(n, d, 128))
    pad = (longest + 127) // 128 * 128
    assert B.workspace_bytes(n, d, p) == 2 * n * pad + 256
    assert B.workspace_bytes(200, d, p) > 0                                   # int16 partials
    ps = B.default_params(rule=B.RULE_SUM)
    assert B.workspace_bytes(n, d, ps) == 2 * n * pad * 4 + 256


def test_host_only_context_refuses_device_calls():
    ctx = B.Brace(4, 1, 100, host_only=True)
    lib = B.lib()
    assert lib.brace_ring_reduce_scatter_step(ctx._ctx, 0, 4096, 100, None) == B.ERR_WORKSPACE
    assert lib.brace_consensus(ctx._ctx, 4096, 4, None) == B.ERR_WORKSPACE
    assert lib.brace_ring_allgather_step(ctx._ctx, 0, 4096, 4, None) == B.ERR_WORKSPACE
    assert lib.brace_aggregate(ctx._ctx, 4096, 100, 4096, 4, None) == B.ERR_WORKSPACE
    assert lib.brace_aggregate(None, 4096, 100, 4096, 4, None) == B.ERR_INVALID_ARG
    assert ctx.last_cuda_error() == 0
    ctx.close()


def test_comm_cost_matches_table1_and_the_oracle_schedule(golden):
    """Table 1 closed forms when n divides d (G = 1); otherwise the per-client
    counts of the oracle's simulated schedule."""
    import numpy as np
    for n, d, m, sc, rar, brace in golden("comm_cost_table1.txt")["rows"]:
        ctx = B.Brace(n, 0, d, B.default_params(granule=1), host_only=True)
        c = ctx.comm_cost(m)
        assert c.sc_bits == sc
        assert c.rar_bits_min == c.rar_bits_max == rar and c.rar_closed_form == rar
        assert c.brace_bits_min == c.brace_bits_max == brace and c.brace_closed_form == brace
        assert c.partial_bits_used == 8
        assert 2 ** c.partial_bits_min >= 2 * n + 1 > 2 ** (c.partial_bits_min - 1)
        ctx.close()
    rng = np.random.default_rng(0)
    for n, d, G in [(5, 23, 1), (7, 1000, 32), (16, 300, 128), (8, 100_000, 128)]:
        U = rng.standard_normal((n, d)).astype(np.float32)
        tr = O.ring_round(U, lam=0, granule=G, keep_states=False)
        ctx = B.Brace(n, 0, d, B.default_params(granule=G), host_only=True)
        c = ctx.comm_cost(32)
        bits = O.sent_bits(tr, 32, O.RULE_SIGN_CONSENSUS)
        assert (c.brace_bits_min, c.brace_bits_max) == (int(bits.min()), int(bits.max()))
        bits = O.sent_bits(tr, 32, O.RULE_SUM)
        assert (c.rar_bits_min, c.rar_bits_max) == (int(bits.min()), int(bits.max()))
        bits = O.sent_bits(tr, 8, O.RULE_SIGN_CONSENSUS)
        assert (c.packed_bits_min, c.packed_bits_max) == (int(bits.min()), int(bits.max()))
        ctx.close()
    big = B.Brace(200, 0, 1000, B.default_params(), host_only=True)
    assert big.comm_cost(32).partial_bits_used == 16 and big.comm_cost(32).partial_bits_min == 9
    assert B.lib().brace_comm_cost(big._ctx, 0, B.Cost()) == B.ERR_INVALID_ARG
    big.close()
