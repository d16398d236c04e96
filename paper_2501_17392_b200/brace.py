"""ctypes binding of the BRACE CUDA library (C ABI in include/brace.h).

Argument marshalling only: every step of the aggregation runs in the CUDA
kernels.  torch is used for device memory and streams.  There is no CPU
fallback: if the compiled library is missing, loading raises.
"""

from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# BRACE_LIBRARY names another build of the same library (the debug build, for instance)
LIB_PATH = os.environ.get("BRACE_LIBRARY") or os.path.join(_PKG, "libbrace.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_BAD_STEP, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(7)
RULE_SIGN_CONSENSUS, RULE_SUM, RULE_MAJORITY_SIGN, RULE_ABS_CONSENSUS = 0, 1, 2, 3
AGG_AUTO, AGG_STEPWISE, AGG_FUSED = 0, 1, 2
STAT_MEDIAN, STAT_TRIMMED_MEAN = 0, 1
ATTACK_NONE, ATTACK_SCALE_OWN, ATTACK_GAUSSIAN, ATTACK_SCALED_MEAN, ATTACK_MEAN_SHIFT, ATTACK_SPARSE_NOISE = range(6)
DRAWS_SUPPLIED, DRAWS_GENERATED = 0, 1
DRAW_UNIFORM, DRAW_NORMAL = 0, 1


class Params(C.Structure):
    _fields_ = [("rule", C.c_int32), ("lam", C.c_float), ("zero_sign", C.c_int32), ("granule", C.c_int32),
                ("mean", C.c_int32), ("agg_mode", C.c_int32)]


class Attack(C.Structure):
    _fields_ = [("kind", C.c_int32), ("scale", C.c_float), ("sigma", C.c_float), ("kappa", C.c_float),
                ("prob", C.c_float), ("h_byz_ids", C.POINTER(C.c_int32)), ("noise", C.c_void_p),
                ("noise_ld", C.c_int64), ("uniform", C.c_void_p), ("uniform_ld", C.c_int64),
                ("draws", C.c_int32), ("round", C.c_uint32), ("seed", C.c_uint64)]


class Cost(C.Structure):
    _fields_ = [("sc_bits", C.c_int64), ("rar_bits_min", C.c_int64), ("rar_bits_max", C.c_int64),
                ("brace_bits_min", C.c_int64), ("brace_bits_max", C.c_int64), ("packed_bits_min", C.c_int64),
                ("packed_bits_max", C.c_int64), ("rar_closed_form", C.c_double), ("brace_closed_form", C.c_double),
                ("partial_bits_used", C.c_int32), ("partial_bits_min", C.c_int32)]


class BraceError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None

# name -> (restype, argtypes); one entry per function declared in include/brace.h
SIGNATURES = {
    "brace_status_string": (C.c_char_p, [C.c_int]),
    "brace_default_params": (C.c_int, [C.POINTER(Params)]),
    "brace_workspace_bytes": (C.c_size_t, [C.c_int32, C.c_int64, C.POINTER(Params)]),
    "brace_init": (C.c_int, [C.POINTER(C.c_void_p), C.c_int32, C.c_int32, C.c_int64, C.POINTER(Params), C.c_void_p,
                             C.c_size_t, C.c_void_p]),
    "brace_destroy": (C.c_int, [C.c_void_p]),
    "brace_segment": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
    "brace_last_cuda_error": (C.c_int, [C.c_void_p]),
    "brace_comm_cost": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(Cost)]),
    "brace_inject_attack": (C.c_int, [C.c_void_p, C.POINTER(Attack), C.c_void_p, C.c_int64, C.c_void_p, C.c_int64,
                                      C.c_void_p]),
    "brace_draw_matrix": (C.c_int, [C.c_int32, C.c_uint64, C.c_uint32, C.c_int32, C.c_int32, C.c_int64, C.c_void_p,
                                    C.c_int64, C.c_float, C.c_float, C.c_void_p]),
    "brace_quantize": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p]),
    "brace_ring_reduce_scatter_step": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p]),
    "brace_consensus": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]),
    "brace_ring_allgather_step": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p]),
    "brace_aggregate": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p]),
    "brace_apply_update": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_float, C.c_void_p]),
    "brace_coordinate_stat": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p,
                                        C.c_void_p]),
    "brace_aggregate_host": (C.c_int, [C.c_void_p, C.POINTER(Attack), C.c_void_p, C.c_int64, C.c_void_p, C.c_int64,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "brace_debug_mailbox": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(C.c_void_p), C.POINTER(C.c_int64),
                                      C.POINTER(C.c_int32), C.POINTER(C.c_int32)]),
    "brace_set_tuning": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32]),
    "brace_debug_status": (C.c_int, [C.POINTER(C.c_int32)]),
    "brace_minmax_rate_probe": (C.c_int, [C.c_int32, C.c_int32, C.c_void_p, C.POINTER(C.c_int64), C.c_void_p]),
    "brace_aggregate_static": (C.c_int, [C.c_int32, C.c_int64, C.POINTER(Params), C.c_void_p, C.c_int64, C.c_void_p,
                                         C.c_int64, C.c_void_p]),
}

STATIC_SCRATCH_BYTES = 8 * 1024 * 1024


def lib() -> C.CDLL:
    """Load the compiled library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2501_17392_b200.build` "
                               "(there is no CPU fallback)")
        handle = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


def status_string(status: int) -> str:
    return lib().brace_status_string(status).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise BraceError(status, where)


def default_params(**over) -> Params:
    p = Params()
    _check(lib().brace_default_params(C.byref(p)), "brace_default_params")
    for k, v in over.items():
        if k == "lambda_":
            k = "lam"
        setattr(p, k, v)
    return p


def workspace_bytes(n: int, d: int, params: Params) -> int:
    return int(lib().brace_workspace_bytes(n, d, C.byref(params)))


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def make_attack(kind: int, *, scale=1.0, sigma=1.0, kappa=3.0, prob=0.1, byz_ids=None, noise=None,
                uniform=None, seed=None, round_idx=0) -> Attack:
    """Build the attack descriptor; keeps the id array alive on the returned object.
    With `seed` given the library draws the attack's random numbers itself from
    (seed, round_idx); otherwise `noise` / `uniform` supply them."""
    a = Attack()
    a.kind, a.scale, a.sigma, a.kappa, a.prob = kind, scale, sigma, kappa, prob
    if seed is not None:
        a.draws, a.seed, a.round = DRAWS_GENERATED, int(seed), int(round_idx)
    if byz_ids is not None:
        arr = (C.c_int32 * len(byz_ids))(*[int(i) for i in byz_ids])
        a._ids_keepalive = arr
        a.h_byz_ids = C.cast(arr, C.POINTER(C.c_int32))
    if noise is not None:
        a._noise_keepalive = noise
        a.noise, a.noise_ld = _ptr(noise), noise.stride(0)
    if uniform is not None:
        a._uniform_keepalive = uniform
        a.uniform, a.uniform_ld = _ptr(uniform), uniform.stride(0)
    return a


def draw_matrix_status(what: int, seed: int, round_idx: int, first_client: int, out: torch.Tensor, d: int,
                       mu=0.0, sigma=1.0, stream=None) -> int:
    return lib().brace_draw_matrix(what, seed, round_idx, first_client, out.shape[0], d, _ptr(out), out.stride(0),
                                   float(mu), float(sigma), _stream(stream))


def draw_matrix(what: int, seed: int, round_idx: int, first_client: int, out: torch.Tensor, d: int, mu=0.0,
                sigma=1.0, stream=None):
    """Fill `out` [rows, ld] with the library's own uniform / normal draws of clients
    first_client .. first_client + rows - 1 (the draws attacks 2 and 5 consume)."""
    _check(draw_matrix_status(what, seed, round_idx, first_client, out, d, mu, sigma, stream), "brace_draw_matrix")


def minmax_rate_probe(blocks: int, iters: int, out: torch.Tensor, stream=None) -> int:
    """Launch the min/max calibration kernel; returns the number of operations it performs."""
    ops = C.c_int64(0)
    _check(lib().brace_minmax_rate_probe(blocks, iters, _ptr(out), C.byref(ops), _stream(stream)),
           "brace_minmax_rate_probe")
    return ops.value


def debug_status():
    """(status, code): code of the first index check that failed in a debug build since the last call."""
    code = C.c_int32(0)
    status = lib().brace_debug_status(C.byref(code))
    return status, code.value


def aggregate_static_status(n: int, d: int, params: Params, updates: torch.Tensor, out: torch.Tensor,
                            stream=None) -> int:
    """brace_aggregate_static: a fused round whose mailboxes live in the library's
    built-in scratch array, for callers that cannot allocate a workspace."""
    return lib().brace_aggregate_static(n, d, C.byref(params), _ptr(updates), updates.stride(0), _ptr(out),
                                        out.stride(0), _stream(stream))


def aggregate_static(n: int, d: int, params: Params, updates: torch.Tensor, out: torch.Tensor, stream=None):
    _check(aggregate_static_status(n, d, params, updates, out, stream), "brace_aggregate_static")


class Brace:
    """One aggregation context: n clients, f Byzantine, d coordinates."""

    def __init__(self, n: int, f: int, d: int, params: Params | None = None, device="cuda", host_only=False,
                 workspace: torch.Tensor | None = None):
        self.n, self.f, self.d = n, f, d
        self.params = params if params is not None else default_params()
        self._ctx = C.c_void_p()
        self.workspace = None
        if host_only:
            ws_ptr, ws_bytes = None, 0
        elif workspace is not None:          # caller-owned uint8 device tensor
            self.workspace = workspace
            ws_ptr, ws_bytes = workspace.data_ptr(), workspace.numel()
        else:
            need = workspace_bytes(n, d, self.params)
            if need == 0:
                # let brace_init report the precise reason
                need = 256
            self.workspace = torch.empty(need, dtype=torch.uint8, device=device)
            ws_ptr, ws_bytes = self.workspace.data_ptr(), need
        _check(lib().brace_init(C.byref(self._ctx), n, f, d, C.byref(self.params), ws_ptr, ws_bytes, None),
               "brace_init")

    # ---- lifetime
    def close(self):
        if self._ctx:
            lib().brace_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- host queries
    def segment(self, j: int):
        b, e = C.c_int64(), C.c_int64()
        _check(lib().brace_segment(self._ctx, j, C.byref(b), C.byref(e)), "brace_segment")
        return b.value, e.value

    def comm_cost(self, m_bits: int) -> Cost:
        cost = Cost()
        _check(lib().brace_comm_cost(self._ctx, m_bits, C.byref(cost)), "brace_comm_cost")
        return cost

    def last_cuda_error(self) -> int:
        return int(lib().brace_last_cuda_error(self._ctx))

    def set_tuning(self, fused_variant=0, fused_grid=0):
        _check(lib().brace_set_tuning(self._ctx, fused_variant, fused_grid), "brace_set_tuning")

    @property
    def out_words(self) -> int:
        return (self.d + 31) // 32

    def new_output(self, out_ld: int | None = None, device="cuda") -> torch.Tensor:
        if self.params.rule == RULE_SUM:
            ld = out_ld or (self.d + 3) // 4 * 4
            return torch.zeros((self.n, ld), dtype=torch.float32, device=device)
        ld = out_ld or (self.out_words + 3) // 4 * 4
        return torch.zeros((self.n, ld), dtype=torch.int32, device=device)

    # ---- device calls (raw status variants end in _status)
    def inject_attack(self, attack: Attack, honest: torch.Tensor, updates: torch.Tensor, stream=None):
        _check(lib().brace_inject_attack(self._ctx, C.byref(attack), _ptr(honest), honest.stride(0), _ptr(updates),
                                         updates.stride(0), _stream(stream)), "brace_inject_attack")

    def quantize(self, updates: torch.Tensor, q: torch.Tensor, stream=None):
        _check(lib().brace_quantize(self._ctx, _ptr(updates), updates.stride(0), _ptr(q), q.stride(0),
                                    _stream(stream)), "brace_quantize")

    def reduce_scatter_step_status(self, step: int, updates: torch.Tensor, stream=None) -> int:
        return lib().brace_ring_reduce_scatter_step(self._ctx, step, _ptr(updates), updates.stride(0),
                                                    _stream(stream))

    def reduce_scatter_step(self, step: int, updates: torch.Tensor, stream=None):
        _check(self.reduce_scatter_step_status(step, updates, stream), "brace_ring_reduce_scatter_step")

    def consensus_status(self, out: torch.Tensor, stream=None) -> int:
        return lib().brace_consensus(self._ctx, _ptr(out), out.stride(0), _stream(stream))

    def consensus(self, out: torch.Tensor, stream=None):
        _check(self.consensus_status(out, stream), "brace_consensus")

    def allgather_step_status(self, step: int, out: torch.Tensor, stream=None) -> int:
        return lib().brace_ring_allgather_step(self._ctx, step, _ptr(out), out.stride(0), _stream(stream))

    def allgather_step(self, step: int, out: torch.Tensor, stream=None):
        _check(self.allgather_step_status(step, out, stream), "brace_ring_allgather_step")

    def aggregate_status(self, updates: torch.Tensor, out: torch.Tensor, stream=None) -> int:
        return lib().brace_aggregate(self._ctx, _ptr(updates), updates.stride(0), _ptr(out), out.stride(0),
                                     _stream(stream))

    def aggregate(self, updates: torch.Tensor, out: torch.Tensor, stream=None):
        _check(self.aggregate_status(updates, out, stream), "brace_aggregate")

    def apply_update_status(self, out: torch.Tensor, weights: torch.Tensor, eta: float, stream=None) -> int:
        return lib().brace_apply_update(self._ctx, _ptr(out), out.stride(0), _ptr(weights), weights.stride(0),
                                        float(eta), _stream(stream))

    def apply_update(self, out: torch.Tensor, weights: torch.Tensor, eta: float, stream=None):
        """Each client's parameter row moves by the aggregate in its output row."""
        _check(self.apply_update_status(out, weights, eta, stream), "brace_apply_update")

    def coordinate_stat_status(self, kind: int, trim: int, updates: torch.Tensor, result: torch.Tensor,
                               stream=None) -> int:
        return lib().brace_coordinate_stat(self._ctx, kind, trim, _ptr(updates), updates.stride(0), _ptr(result),
                                           _stream(stream))

    def coordinate_stat(self, kind: int, trim: int, updates: torch.Tensor, result: torch.Tensor, stream=None):
        """Coordinate-wise median / trimmed mean of the n rows into one float32 vector."""
        _check(self.coordinate_stat_status(kind, trim, updates, result, stream), "brace_coordinate_stat")

    def aggregate_host(self, attack: Attack | None, h_updates: torch.Tensor, h_out: torch.Tensor,
                       d_updates: torch.Tensor, d_out: torch.Tensor, d_noise=None, d_uniform=None, stream=None):
        """Host-buffer round: h_updates / h_out (and attack.noise / uniform) are CPU
        tensors, ideally pinned; the d_* tensors are device staging of the same shapes."""
        assert h_updates.stride(0) == d_updates.stride(0) and h_out.stride(0) == d_out.stride(0)
        _check(lib().brace_aggregate_host(self._ctx, C.byref(attack) if attack is not None else None,
                                          _ptr(h_updates), h_updates.stride(0), _ptr(h_out), h_out.stride(0),
                                          _ptr(d_updates), _ptr(d_noise), _ptr(d_uniform), _ptr(d_out),
                                          _stream(stream)), "brace_aggregate_host")

    def debug_mailbox(self, client: int, hops_back: int = 0):
        """(device pointer, length, sub-vector id, entry bytes) of a client's mailbox."""
        p, ln, seg, eb = C.c_void_p(), C.c_int64(), C.c_int32(), C.c_int32()
        _check(lib().brace_debug_mailbox(self._ctx, client, hops_back, C.byref(p), C.byref(ln), C.byref(seg),
                                         C.byref(eb)), "brace_debug_mailbox")
        return p.value, ln.value, seg.value, eb.value

    def mailbox_tensor(self, client: int, hops_back: int = 0) -> tuple[int, torch.Tensor]:
        """(sub-vector id, copy of the mailbox contents as a CPU int64/float32 tensor)."""
        p, ln, seg, eb = self.debug_mailbox(client, hops_back)
        off = p - self.workspace.data_ptr()
        raw = self.workspace[off: off + ln * eb]
        dt = {1: torch.int8, 2: torch.int16, 4: torch.float32}[eb]
        return seg, raw.view(dt).cpu()
