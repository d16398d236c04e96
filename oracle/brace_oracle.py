"""CPU oracle for BRACE ring aggregation.  TEST INFRASTRUCTURE ONLY.

This module is a plain, slow, by-eye-checkable numpy restatement of what the
paper "Byzantine-Robust Federated Learning over Ring-All-Reduce Distributed
Computing" (BRACE) computes in one aggregation round.  It exists to check the
CUDA library; it is never part of the product path.  Only the test-suite, the
smoke check and the benchmark's CPU-baseline / reference legs may import it.
It shares no code with the CUDA library and imports nothing from it.

Every function names the passage of the paper it follows.  Where the method
has an exact plain definition (Eq. (1): a threshold on an integer sum) the
oracle is that definition; where the paper describes a procedure (the ring
schedule of Section 2.2 and Section 3) the oracle performs the procedure hop
by hop on literal per-client arrays, snapshotting every message of a hop
before applying any of them, exactly as n concurrent clients would.

Readings of points the paper leaves open (all are parameters, defaults below):
  * sign(0) = 0, sign(NaN) = 0, sign(+-Inf) = +-1 (``zero_sign`` in {-1,0,+1}
    maps exact zeros elsewhere); Section 3 Phase I only says "element-wise sign".
  * lambda may be any finite real; the sign-sum is an integer, so
    ``S > lambda`` is evaluated as ``S > floor(lambda)``; ties give -1 as
    Eq. (1) prints.
  * "n roughly equal-sized sub-vectors" (Section 2.2): sub-vector boundaries
    fall on multiples of a granule of G coordinates, see ``partition``.
  * ring direction and hop -> sub-vector map: fixed by the three-client worked
    example of Section 2.2 (0-based: at share-reduce hop s client c sends
    sub-vector (c - s) mod n to client (c + 1) mod n; after n-1 hops client c
    owns sub-vector (c + 1) mod n; at share-only hop t client c sends
    sub-vector (c + 1 - t) mod n).

Parity status: every function here is pinned by tests/test_oracle_pins.py
(printed worked example, closed forms, invariants, brute force); none is
"parity unpinned".
"""

from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

RULE_SIGN_CONSENSUS = 0  # BRACE, Section 3, Eq. (1)
RULE_SUM = 1             # plain ring-all-reduce, Section 2.2
RULE_MAJORITY_SIGN = 2   # signSGD with majority vote over the ring (Section 5.2)
RULE_ABS_CONSENSUS = 3   # RLR-style test on |sign-sum| over the ring (Section 5.2)
SIGN_RULES = (RULE_SIGN_CONSENSUS, RULE_MAJORITY_SIGN, RULE_ABS_CONSENSUS)

ATTACK_SCALE_OWN = 1     # b_i = a * h_i
ATTACK_GAUSSIAN = 2      # b_i = sigma * z_i
ATTACK_SCALED_MEAN = 3   # b_i = a * mean_honest
ATTACK_MEAN_SHIFT = 4    # b_i = mean_honest - kappa * std_honest
ATTACK_SPARSE_NOISE = 5  # b_i[k] = sigma * z_i[k] if u_i[k] < p else 0


# --------------------------------------------------------------------------
# Section 2.2: "splitting its gradient into n roughly equal-sized sub-vectors"
# --------------------------------------------------------------------------
def partition(n: int, d: int, granule: int = 128):
    """Sub-vector j covers coordinates [begin_j, end_j).

    The d coordinates are grouped into Q = ceil(d / G) granules of G
    coordinates (the last one possibly short); sub-vector j takes granules
    floor(j*Q/n) .. floor((j+1)*Q/n) - 1.  G = 1 is the balanced split of d
    into n parts.  Sub-vectors may be empty when d < n*G.
    """
    if n < 2 or d < 1 or granule < 1:
        raise ValueError("need n >= 2, d >= 1, granule >= 1")
    q = -(-d // granule)
    bounds = []
    for j in range(n):
        b = min(granule * ((j * q) // n), d)
        e = min(granule * (((j + 1) * q) // n), d)
        bounds.append((b, e))
    return bounds


# --------------------------------------------------------------------------
# Section 3, Phase I (Quantization): element-wise sign
# --------------------------------------------------------------------------
def sgn(x: np.ndarray, zero_sign: int = 0) -> np.ndarray:
    """Element-wise sign as int32: (x > 0) - (x < 0); exact zeros and NaN give
    ``zero_sign`` for zeros and 0 for NaN."""
    x = np.asarray(x)
    s = (x > 0).astype(np.int32) - (x < 0).astype(np.int32)
    if zero_sign != 0:
        s = np.where(x == 0, np.int32(zero_sign), s)
    return s.astype(np.int32)


def lambda_int(lam: float, n: int) -> int:
    """Integer threshold equivalent to the real lambda of Eq. (1): for integer S,
    S > lambda  <=>  S > floor(lambda); clamped to [-n-1, n] (beyond that range
    the comparison is constant)."""
    if not math.isfinite(lam):
        raise ValueError("lambda must be finite")
    return int(max(-n - 1, min(n, math.floor(lam))))


# --------------------------------------------------------------------------
# Section 3, Phase III: the map applied to the integer sign-sum S
# --------------------------------------------------------------------------
def consensus_map(total: np.ndarray, rule: int, lam: float, n: int) -> np.ndarray:
    """+-1 vector from the sign-sums.

    RULE_SIGN_CONSENSUS  Eq. (1): +1 if S > lambda else -1.
    RULE_MAJORITY_SIGN   Section 5.2, signSGD carried over the ring: the sign of
                         S; the paper does not say what S = 0 gives, here -1.
    RULE_ABS_CONSENSUS   Section 5.2, the RLR-style test: "the absolute value of
                         the sum", positive and negative agreement alike:
                         +1 if |S| > lambda else -1 (strictness as in Eq. (1)).
    """
    if rule == RULE_SIGN_CONSENSUS:
        return np.where(total > lambda_int(lam, n), 1, -1).astype(np.int8)
    if rule == RULE_MAJORITY_SIGN:
        return np.where(total > 0, 1, -1).astype(np.int8)
    if rule == RULE_ABS_CONSENSUS:
        return np.where(np.abs(total) > lambda_int(lam, n), 1, -1).astype(np.int8)
    raise ValueError("not a sign rule")


# --------------------------------------------------------------------------
# Section 3, Phase III, Eq. (1): the aggregation rule as a plain definition
# --------------------------------------------------------------------------
def gar_direct(updates: np.ndarray, lam: float, zero_sign: int = 0, rule: int = RULE_SIGN_CONSENSUS) -> np.ndarray:
    """GAR(g_1..g_n)[k] = +1 if sum_i sign(g_i[k]) > lambda else -1 (Eq. (1));
    other sign rules swap the final map, see ``consensus_map``.

    updates: [n, d].  Returns int8 [d] with entries in {-1, +1}.
    """
    updates = np.asarray(updates)
    n = updates.shape[0]
    total = np.zeros(updates.shape[1], dtype=np.int32)
    for i in range(n):
        total = total + sgn(updates[i], zero_sign)
    return consensus_map(total, rule, lam, n)


def sign_sum_direct(updates: np.ndarray, zero_sign: int = 0) -> np.ndarray:
    """S[k] = sum_i sign(g_i[k]) (the quantity thresholded in Eq. (1))."""
    updates = np.asarray(updates)
    total = np.zeros(updates.shape[1], dtype=np.int32)
    for i in range(updates.shape[0]):
        total = total + sgn(updates[i], zero_sign)
    return total


# --------------------------------------------------------------------------
# Output representation: 1 bit per dimension (Section 3, cost paragraph)
# --------------------------------------------------------------------------
def pack_bits(pm1: np.ndarray, words: int | None = None) -> np.ndarray:
    """Pack a {-1,+1} vector into uint32 words: coordinate k is bit (k mod 32),
    least significant first, of word (k div 32); +1 -> 1, -1 -> 0; padding 0."""
    pm1 = np.asarray(pm1)
    d = pm1.shape[0]
    nwords = -(-d // 32) if words is None else words
    out = np.zeros(nwords, dtype=np.uint32)
    for k in range(d):
        if pm1[k] > 0:
            out[k // 32] |= np.uint32(1) << np.uint32(k % 32)
    return out


def pack_bits_fast(pm1: np.ndarray, words: int | None = None) -> np.ndarray:
    """Same mapping as ``pack_bits`` through numpy's packbits (little bit order);
    tests check the two agree."""
    pm1 = np.asarray(pm1)
    d = pm1.shape[0]
    nwords = -(-d // 32) if words is None else words
    bits = np.zeros(nwords * 32, dtype=np.uint8)
    bits[:d] = pm1 > 0
    return np.packbits(bits, bitorder="little").view("<u4").astype(np.uint32)


# --------------------------------------------------------------------------
# Sections 2.2 and 3: the ring procedure, hop by hop
# --------------------------------------------------------------------------
@dataclass
class RingTrace:
    """Everything a round of the ring leaves behind.

    outputs      [n, d]  what each client holds after Share-Only
                         (int8 +-1 for BRACE, float32 for SUM)
    rs_states    list over share-reduce hops s of a list over clients r of
                 (sub-vector id, copy of client r's reduced partial for that
                 sub-vector after hop s)
    owned        list over clients c of (sub-vector id, fully reduced partial)
                 after the last share-reduce hop
    rs_sent      [n] coordinates each client sent during share-reduce
    ag_sent      [n] coordinates each client sent during share-only
    bounds       the partition used
    """
    outputs: np.ndarray
    rs_states: list = field(default_factory=list)
    owned: list = field(default_factory=list)
    rs_sent: np.ndarray | None = None
    ag_sent: np.ndarray | None = None
    bounds: list = field(default_factory=list)
    ag_states: list = field(default_factory=list)


def ring_round(updates: np.ndarray, rule: int = RULE_SIGN_CONSENSUS, lam: float = 0.0,
               zero_sign: int = 0, granule: int = 128, mean: bool = False,
               keep_states: bool = True) -> RingTrace:
    """One aggregation round on literal per-client arrays.

    BRACE (rule = RULE_SIGN_CONSENSUS), Section 3:
      Phase I   every client replaces its vector by its element-wise sign;
      Phase II  share-reduce: n-1 hops; at hop s client c sends its current
                sub-vector (c - s) mod n downstream, the receiver adds it to its
                own copy of that sub-vector;
      Phase III the owner of each fully reduced sub-vector thresholds it with
                lambda (Eq. (1));
      Phase IV  share-only: n-1 hops; at hop t client c sends sub-vector
                (c + 1 - t) mod n downstream, the receiver overwrites.
    Plain RAR (rule = RULE_SUM), Section 2.2: same Phases II and IV on the raw
    float32 vectors (additions in float32, in the order the ring performs
    them); Phase III is the identity, or division by n when ``mean`` is set.
    """
    updates = np.asarray(updates)
    n, d = updates.shape
    bounds = partition(n, d, granule)

    # Phase I (BRACE) / local copies (SUM): one full-length working vector per client
    if rule in SIGN_RULES:
        work = [sgn(updates[c], zero_sign) for c in range(n)]
    elif rule == RULE_SUM:
        work = [np.array(updates[c], dtype=np.float32, copy=True) for c in range(n)]
    else:
        raise ValueError("unknown rule")

    trace = RingTrace(outputs=np.empty(0), bounds=bounds)
    rs_sent = np.zeros(n, dtype=np.int64)
    ag_sent = np.zeros(n, dtype=np.int64)

    # Phase II: Share-Reduce
    for s in range(n - 1):
        messages = []
        for c in range(n):                      # all clients send at once: snapshot first
            j = (c - s) % n
            b, e = bounds[j]
            messages.append((c, j, work[c][b:e].copy()))
            rs_sent[c] += e - b
        states = []
        for c, j, payload in messages:          # then every receiver reduces
            r = (c + 1) % n
            b, e = bounds[j]
            work[r][b:e] = payload + work[r][b:e]
        if keep_states:
            for r in range(n):
                j = (r - 1 - s) % n
                b, e = bounds[j]
                states.append((j, work[r][b:e].copy()))
            trace.rs_states.append(states)

    # ownership after n-1 hops: client c holds the reduced sub-vector (c+1) mod n
    for c in range(n):
        j = (c + 1) % n
        b, e = bounds[j]
        trace.owned.append((j, work[c][b:e].copy()))

    # Phase III: Consensus (BRACE) / identity or mean (SUM), local to the owner
    if rule in SIGN_RULES:
        result = [np.zeros(d, dtype=np.int8) for _ in range(n)]
        for c in range(n):
            j = (c + 1) % n
            b, e = bounds[j]
            result[c][b:e] = consensus_map(work[c][b:e], rule, lam, n)
    else:
        result = [np.zeros(d, dtype=np.float32) for _ in range(n)]
        for c in range(n):
            j = (c + 1) % n
            b, e = bounds[j]
            seg = work[c][b:e]
            result[c][b:e] = (seg / np.float32(n)) if mean else seg

    # Phase IV: Share-Only
    for t in range(n - 1):
        messages = []
        for c in range(n):
            j = (c + 1 - t) % n
            b, e = bounds[j]
            messages.append((c, j, result[c][b:e].copy()))
            ag_sent[c] += e - b
        for c, j, payload in messages:
            r = (c + 1) % n
            b, e = bounds[j]
            result[r][b:e] = payload
        if keep_states:
            trace.ag_states.append([row.copy() for row in result])

    trace.outputs = np.stack(result)
    trace.rs_sent = rs_sent
    trace.ag_sent = ag_sent
    return trace


def sum_direct_f64(updates: np.ndarray) -> np.ndarray:
    """sum_i g_i in float64 (Section 2.2: what every client holds after RAR)."""
    updates = np.asarray(updates)
    acc = np.zeros(updates.shape[1], dtype=np.float64)
    for i in range(updates.shape[0]):
        acc = acc + updates[i].astype(np.float64)
    return acc


# --------------------------------------------------------------------------
# Section 5.1: the server-side coordinate-wise rules BRACE is compared with
# --------------------------------------------------------------------------
def coordinate_median(updates: np.ndarray) -> np.ndarray:
    """Coordinate-wise median of the n client values: the middle one of the n
    sorted values, for even n the mean of the two middle ones (float64), rounded
    to float32."""
    srt = np.sort(np.asarray(updates, dtype=np.float32), axis=0)
    n = srt.shape[0]
    if n % 2 == 1:
        return srt[n // 2]
    lo, hi = srt[n // 2 - 1].astype(np.float64), srt[n // 2].astype(np.float64)
    with np.errstate(invalid="ignore"):
        return (0.5 * (lo + hi)).astype(np.float32)


def coordinate_trimmed_mean(updates: np.ndarray, trim: int) -> np.ndarray:
    """Coordinate-wise trimmed mean: per coordinate drop the ``trim`` smallest and
    the ``trim`` largest of the n values and average the rest (summed in float64
    in ascending order, one rounding to float32)."""
    srt = np.sort(np.asarray(updates, dtype=np.float32), axis=0)
    n = srt.shape[0]
    if trim < 0 or 2 * trim >= n:
        raise ValueError("need 0 <= 2*trim < n")
    acc = np.zeros(srt.shape[1], dtype=np.float64)
    with np.errstate(invalid="ignore"):                 # +Inf and -Inf in one column give NaN, as they should
        for i in range(trim, n - trim):
            acc = acc + srt[i].astype(np.float64)
    return (acc / np.float64(n - 2 * trim)).astype(np.float32)


# --------------------------------------------------------------------------
# The model update that follows a round
# --------------------------------------------------------------------------
def apply_update(weights: np.ndarray, outputs: np.ndarray, eta: float, rule: int, mean: bool = False) -> np.ndarray:
    """Per-client parameter update, in float64.

    Plain RAR (Section 2.2): w_i <- w_i - (eta / n) * sum_j g_j, each client on
    its own copy; ``outputs`` are the rows the ring left (the sum, or the mean
    when ``mean``).  Sign rules (Appendix A, update rule): w <- w - eta * (2 I - 1)
    = w - eta * GAR, no 1/n.  weights, outputs: [n, d].
    """
    w = np.asarray(weights, dtype=np.float64)
    g = np.asarray(outputs, dtype=np.float64)
    n = w.shape[0]
    eta64 = np.float64(np.float32(eta))
    if rule == RULE_SUM:
        factor = eta64 if mean else eta64 / np.float64(n)
        return w - factor * g
    return w - eta64 * g


# --------------------------------------------------------------------------
# Section 2.2 / Section 3 / Table 1: bits each client sends per round
# --------------------------------------------------------------------------
def sent_bits(trace: RingTrace, m_bits: int, rule: int) -> np.ndarray:
    """Bits sent per client: share-reduce moves m bits per coordinate; share-only
    moves 1 bit per coordinate under BRACE and m bits under plain RAR."""
    ag_width = 1 if rule in SIGN_RULES else m_bits
    return trace.rs_sent * m_bits + trace.ag_sent * ag_width


def cost_sc(m, n, d):      # Section 2.2, Table 1
    return m * n * d


def cost_rar(m, n, d):     # Section 2.2, Table 1 (exact rational kept as a pair)
    return 2 * m * d * (n - 1), n


def cost_brace(m, n, d):   # Section 3, Table 1
    return d * (n - 1) * (m + 1), n


# --------------------------------------------------------------------------
# Random draws of the attacks that consume randomness (the Gaussian attack the
# paper names in Section 5.1, and the sparse-noise alteration).  The paper gives
# no generator; the library draws from a counter-based one so that a draw is a
# pure function of (seed, round, client, coordinate, stream) and the CPU and GPU
# sides can each implement it from its published definition: Philox4x32 with 10
# rounds (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as
# 1, 2, 3", SC'11).  This is this module's own implementation of that
# definition; tests pin it to the known-answer vectors published with it.
# --------------------------------------------------------------------------
PHILOX_M0 = 0xD2511F53   # round multipliers
PHILOX_M1 = 0xCD9E8D57
PHILOX_W0 = 0x9E3779B9   # key increments per round (golden ratio, sqrt(3) - 1)
PHILOX_W1 = 0xBB67AE85

STREAM_UNIFORM = 0       # one 32-bit word per coordinate -> uniform in [0, 1)
STREAM_NORMAL = 1        # two words per coordinate pair -> two standard normals (Box-Muller)


def philox4x32_10(counter, key):
    """The Philox4x32-10 bijection on arrays of counters.

    counter: four uint32 arrays (broadcastable to one shape), key: two uint32
    values/arrays.  Returns four uint32 arrays.  One round maps
    (c0, c1, c2, c3), (k0, k1) to
    (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2), hi(M0*c0) ^ c3 ^ k1, lo(M0*c0));
    the key advances by (W0, W1) between rounds.
    """
    c0, c1, c2, c3 = [np.asarray(c, dtype=np.uint64) for c in counter]
    k0, k1 = [np.asarray(k, dtype=np.uint64) for k in key]
    mask = np.uint64(0xFFFFFFFF)
    for _ in range(10):
        p0 = np.uint64(PHILOX_M0) * c0          # 32 x 32 -> 64 bits, no overflow in uint64
        p1 = np.uint64(PHILOX_M1) * c2
        n0 = (p1 >> np.uint64(32)) ^ c1 ^ k0
        n1 = p1 & mask
        n2 = (p0 >> np.uint64(32)) ^ c3 ^ k1
        n3 = p0 & mask
        c0, c1, c2, c3 = n0, n1, n2, n3
        k0 = (k0 + np.uint64(PHILOX_W0)) & mask
        k1 = (k1 + np.uint64(PHILOX_W1)) & mask
    return [c.astype(np.uint32) for c in (c0, c1, c2, c3)]


def draw_words(seed: int, round_idx: int, client: int, stream: int, d: int, start: int = 0) -> np.ndarray:
    """The raw 32-bit words of coordinates start .. start + d - 1 (start a multiple
    of 4) of one client's row of one stream.

    Coordinates are served four at a time: block q = k div 4 is one Philox call
    with key = (seed mod 2^32, seed div 2^32) and counter
    (q mod 2^32, q div 2^32, client, round * 256 + stream); word k mod 4 of the
    result belongs to coordinate k.  round < 2^24, stream < 256.
    """
    if not (0 <= seed < 1 << 64 and 0 <= round_idx < 1 << 24 and 0 <= stream < 256 and 0 <= client < 1 << 32):
        raise ValueError("seed, round, client or stream out of range")
    if start < 0 or start % 4:
        raise ValueError("start must be a non-negative multiple of 4")
    nblk = -(-d // 4)
    q = np.arange(nblk, dtype=np.uint64) + np.uint64(start // 4)
    words = philox4x32_10(
        (q & np.uint64(0xFFFFFFFF), q >> np.uint64(32), np.uint64(client), np.uint64(round_idx * 256 + stream)),
        (np.uint64(seed & 0xFFFFFFFF), np.uint64(seed >> 32)))
    return np.stack(words, axis=1).reshape(-1)[:d]


def draw_uniform(seed: int, round_idx: int, client: int, d: int, start: int = 0) -> np.ndarray:
    """float32 [d], uniform on the 2^24 multiples of 2^-24 in [0, 1): the top 24
    bits of the coordinate's word of STREAM_UNIFORM, times 2^-24 (exact)."""
    w = draw_words(seed, round_idx, client, STREAM_UNIFORM, d, start)
    return ((w >> np.uint32(8)).astype(np.float64) * 2.0 ** -24).astype(np.float32)


def _cospi_sinpi(x: np.ndarray):
    """cos(pi x), sin(pi x) for float64 x in [0, 2) with the argument reduced
    exactly first (x is a multiple of 2^-23 here), so that the zeros of both
    functions come out as exact zeros."""
    n = np.rint(2.0 * x)                       # nearest multiple of 1/2
    r = x - 0.5 * n                            # exact; |r| <= 1/4
    c, s = np.cos(np.pi * r), np.sin(np.pi * r)
    quad = n.astype(np.int64) & 3
    cos_out = np.choose(quad, [c, -s, -c, s])
    sin_out = np.choose(quad, [s, c, -s, -c])
    return cos_out, sin_out


def draw_normal(seed: int, round_idx: int, client: int, d: int, start: int = 0) -> np.ndarray:
    """float32 [d] standard normals by the Box-Muller transform, evaluated in
    float64 and rounded once.  Coordinates 2p and 2p+1 share the words (a, b) of
    STREAM_NORMAL at those two coordinates: u1 = ((a >> 8) + 1) / 2^24 in (0, 1],
    u2 = (b >> 8) / 2^24 in [0, 1), radius = sqrt(-2 ln u1);
    z[2p] = radius * cos(2 pi u2), z[2p+1] = radius * sin(2 pi u2)."""
    dp = d + (d & 1)
    w = draw_words(seed, round_idx, client, STREAM_NORMAL, dp, start).reshape(-1, 2)
    u1 = ((w[:, 0] >> np.uint32(8)).astype(np.float64) + 1.0) * 2.0 ** -24
    u2 = (w[:, 1] >> np.uint32(8)).astype(np.float64) * 2.0 ** -24
    radius = np.sqrt(-2.0 * np.log(u1))
    c, s = _cospi_sinpi(2.0 * u2)
    z = np.stack([radius * c, radius * s], axis=1).reshape(-1)[:d]
    return z.astype(np.float32)


def attack_draws(kind: int, seed: int, round_idx: int, byz_ids, d: int, start: int = 0):
    """(noise, uniform) matrices [len(byz_ids), d] an attack of this kind consumes
    when the library draws for itself: row b holds client byz_ids[b]'s draws for
    coordinates start .. start + d - 1."""
    noise = uniform = None
    if kind in (ATTACK_GAUSSIAN, ATTACK_SPARSE_NOISE):
        noise = np.stack([draw_normal(seed, round_idx, int(i), d, start) for i in byz_ids])
    if kind == ATTACK_SPARSE_NOISE:
        uniform = np.stack([draw_uniform(seed, round_idx, int(i), d, start) for i in byz_ids])
    return noise, uniform


# --------------------------------------------------------------------------
# Section 3 (threat model): Byzantine clients alter their vectors before the
# ring starts.  The five synthetic alterations of the benchmark workloads.
# --------------------------------------------------------------------------
def inject_attack(kind: int, honest: np.ndarray, byz_ids, *, scale: float = 1.0,
                  sigma: float = 1.0, kappa: float = 3.0, prob: float = 0.1,
                  noise: np.ndarray | None = None,
                  uniform: np.ndarray | None = None) -> np.ndarray:
    """Return the update matrix the ring will see: honest rows unchanged,
    Byzantine rows replaced.  Arithmetic in float64, one final rounding to
    float32.  ``noise`` / ``uniform`` are [len(byz_ids), d] arrays of standard
    normal / uniform[0,1) draws supplied by the caller (row b belongs to
    byz_ids[b]).  Statistics over honest rows accumulate in increasing client id.
    """
    honest = np.asarray(honest, dtype=np.float32)
    n, d = honest.shape
    byz_ids = [int(i) for i in byz_ids]
    byz = set(byz_ids)
    good = [i for i in range(n) if i not in byz]
    out = honest.copy()
    if not byz_ids:
        return out

    if kind == ATTACK_SCALE_OWN:
        for i in byz_ids:
            out[i] = (np.float64(np.float32(scale)) * honest[i].astype(np.float64)).astype(np.float32)
    elif kind == ATTACK_GAUSSIAN:
        for b, i in enumerate(byz_ids):
            out[i] = (np.float64(np.float32(sigma)) * noise[b].astype(np.float64)).astype(np.float32)
    elif kind in (ATTACK_SCALED_MEAN, ATTACK_MEAN_SHIFT):
        m = len(good)
        if m == 0:
            raise ValueError("no honest client to take statistics over")
        total = np.zeros(d, dtype=np.float64)
        for i in good:
            total = total + honest[i].astype(np.float64)
        mean = total / np.float64(m)
        if kind == ATTACK_SCALED_MEAN:
            vec = np.float64(np.float32(scale)) * mean
        else:
            sq = np.zeros(d, dtype=np.float64)
            for i in good:
                dev = honest[i].astype(np.float64) - mean
                sq = sq + dev * dev
            std = np.sqrt(sq / np.float64(m))          # population std (ddof = 0)
            vec = mean - np.float64(np.float32(kappa)) * std
        vec32 = vec.astype(np.float32)
        for i in byz_ids:
            out[i] = vec32
    elif kind == ATTACK_SPARSE_NOISE:
        p32 = np.float32(prob)
        for b, i in enumerate(byz_ids):
            val = (np.float64(np.float32(sigma)) * noise[b].astype(np.float64)).astype(np.float32)
            out[i] = np.where(uniform[b].astype(np.float32) < p32, val, np.float32(0.0))
    else:
        raise ValueError("unknown attack kind")
    return out
