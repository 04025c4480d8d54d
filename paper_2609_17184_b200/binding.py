"""ctypes binding of include/loopspec.h (argument marshalling only)."""
import ctypes as C
import os

import numpy as np

from . import build as _build

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libloopspec.so")

EXPORTS = ["loopspec_workspace_bytes", "loopspec_init", "loopspec_prefill", "loopspec_step", "loopspec_verify",
           "loopspec_decode", "loopspec_vanilla_decode", "loopspec_pick_depths", "loopspec_fit_envelope", "loopspec_max_branches",
           "loopspec_get_stats", "loopspec_get_commits", "loopspec_get_row_trace", "loopspec_debug_logits",
           "loopspec_launches_per_step", "loopspec_decode_paths", "loopspec_debug_drop_tile", "loopspec_time_kernel", "loopspec_linear_scratch_bytes", "loopspec_op_linear",
           "loopspec_op_linear_static", "loopspec_linear_tc_scratch_bytes", "loopspec_op_linear_tc", "loopspec_time_linear_tc",
           "loopspec_last_error", "loopspec_destroy"]

STATUS = {0: "OK", -1: "EINVAL", -2: "ESTATE", -3: "ECAPACITY", -4: "ECUDA", -5: "ETIMEOUT", -6: "EUNSUPPORTED"}


class LoopSpecError(RuntimeError):
    def __init__(self, code, msg=""):
        super().__init__(f"loopspec: {STATUS.get(code, code)} {msg}".strip())
        self.code = code
        self.status = STATUS.get(code, str(code))


class Model(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("vocab", "hidden", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "n_prelude",
                                         "n_recurrent", "n_coda", "R", "weight_dtype", "tied_lm_head")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)]


class Sched(C.Structure):
    _fields_ = [("d1", C.c_int32), ("d2", C.c_int32), ("alpha", C.c_float), ("beta", C.c_float), ("gate", C.c_int32),
                ("residual_q2", C.c_int32), ("temperature", C.c_float), ("seed", C.c_uint64), ("max_seqs", C.c_int32),
                ("max_ctx", C.c_int32), ("max_prefill_rows", C.c_int32), ("top_k", C.c_int32), ("top_p", C.c_float),
                ("measure_tv", C.c_int32), ("mask_first", C.c_int32), ("prefill_skinny", C.c_int32)]


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p), ("adapter", C.c_void_p),
                ("layer_ptrs", C.POINTER(C.c_void_p))]


class Commit(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("seq", "n_committed", "token", "source", "accepted1", "accepted2", "gate_open",
                                         "step")]


class Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("steps", "n_decode", "n_accept1", "n_accept2", "n_restart", "gate_evals",
                                         "gate_opens", "rows_total", "rows_max", "readout_rows_total")] + \
               [("gamma", C.c_double), ("tv_d1", C.c_double), ("tv_d2", C.c_double), ("tv_n1", C.c_int64), ("tv_n2", C.c_int64)]


def _load():
    if not os.path.exists(_LIB_PATH) or _build.needs_build():
        try:
            _build.build()
        except Exception as e:  # no silent fallback: the CUDA library is the product
            if not os.path.exists(_LIB_PATH):
                raise ImportError(f"libloopspec.so is missing and could not be built: {e}") from e
    lib = C.CDLL(_LIB_PATH)
    P, I, V = C.POINTER, C.c_int32, C.c_void_p
    lib.loopspec_workspace_bytes.restype = C.c_size_t
    lib.loopspec_workspace_bytes.argtypes = [P(Model), P(Sched)]
    lib.loopspec_fit_envelope.argtypes = [P(C.c_double), I, P(C.c_double), P(C.c_double)]
    lib.loopspec_init.argtypes = [P(Model), P(Sched), P(Weights), V, C.c_size_t, V, P(V)]
    lib.loopspec_prefill.argtypes = [V, I, P(I), I, P(I)]
    lib.loopspec_step.argtypes = [V, P(I), P(I)]
    lib.loopspec_verify.argtypes = [V, P(Commit), I, P(I)]
    lib.loopspec_decode.argtypes = [V, I, P(I)]
    lib.loopspec_vanilla_decode.argtypes = [V, I, P(I)]
    lib.loopspec_pick_depths.argtypes = [C.c_float, C.c_float, I, P(C.c_double), P(C.c_double), P(I), P(I)]
    lib.loopspec_max_branches.argtypes = [I, I, I]
    lib.loopspec_max_branches.restype = I
    lib.loopspec_get_stats.argtypes = [V, P(Stats)]
    lib.loopspec_get_commits.argtypes = [V, I, P(Commit), I, P(I)]
    lib.loopspec_get_row_trace.argtypes = [V, P(I), I, P(I)]
    lib.loopspec_debug_logits.argtypes = [V, I, I, P(C.c_float)]
    lib.loopspec_launches_per_step.argtypes = [V, P(I)]
    lib.loopspec_decode_paths.argtypes = [V, P(I), P(I)]
    lib.loopspec_debug_drop_tile.argtypes = [V, I, I]
    lib.loopspec_time_kernel.argtypes = [V, I, I, I, P(C.c_float), P(C.c_double)]
    lib.loopspec_linear_scratch_bytes.restype = C.c_size_t
    lib.loopspec_linear_scratch_bytes.argtypes = [I, I, I]
    lib.loopspec_op_linear.argtypes = [V, I, V, V, I, I, I, V, C.c_size_t, V]
    lib.loopspec_linear_tc_scratch_bytes.restype = C.c_size_t
    lib.loopspec_linear_tc_scratch_bytes.argtypes = [I, I, I]
    lib.loopspec_op_linear_tc.argtypes = [V, V, V, I, I, I, V, C.c_size_t, V]
    lib.loopspec_time_linear_tc.argtypes = [C.POINTER(V), I, V, I, I, I, V, C.c_size_t, I, C.POINTER(C.c_float), V]
    lib.loopspec_op_linear_static.argtypes = [V, I, V, V, I, I, I, V]
    lib.loopspec_last_error.restype = C.c_char_p
    lib.loopspec_last_error.argtypes = [V]
    lib.loopspec_destroy.argtypes = [V]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if fn.restype is C.c_int:  # default restype: the status code
            fn.restype = C.c_int
    return lib


lib = _load()


def pick_depths(alpha, beta, R):
    a, b, x, y = C.c_double(), C.c_double(), C.c_int32(), C.c_int32()
    rc = lib.loopspec_pick_depths(alpha, beta, R, C.byref(a), C.byref(b), C.byref(x), C.byref(y))
    if rc:
        raise LoopSpecError(rc)
    return a.value, b.value, x.value, y.value


def fit_envelope(tv):
    """(alpha, beta) of the power-law envelope over a measured TV profile tv[r-1] = TV(p_r, p_R)."""
    arr = (C.c_double * len(tv))(*[float(x) for x in tv])
    a, b = C.c_double(), C.c_double()
    rc = lib.loopspec_fit_envelope(arr, len(tv), C.byref(a), C.byref(b))
    if rc:
        raise LoopSpecError(rc)
    return a.value, b.value


def max_branches(R, d1, d2):
    return lib.loopspec_max_branches(R, d1, d2)


def upload_weights(shape, w, device="cuda"):
    """numpy float32 arrays (see workloads.make_weights) -> torch tensors on the device in the model's dtype."""
    import torch
    dt = torch.bfloat16 if shape.weight_dtype == "bf16" else torch.float32
    out = {}
    for k, a in w.items():
        t = torch.from_numpy(np.ascontiguousarray(a))
        out[k] = t.to(device=device, dtype=torch.float32 if a.ndim == 1 else dt).contiguous()
    return out


def linear_scratch_bytes(M, N, K):
    return lib.loopspec_linear_scratch_bytes(M, N, K)


def linear(W, x, scratch=None):
    """y = x @ W.T through the weight-streaming kernel.  W [N,K] bf16 or fp32, x [M,K] fp32 (cuda tensors)."""
    import torch
    M, K = x.shape
    N = W.shape[0]
    need = linear_scratch_bytes(M, N, K)
    if need == 0:
        raise LoopSpecError(-1, "unsupported linear shape")
    if scratch is None:
        scratch = torch.zeros(need, dtype=torch.uint8, device=x.device)
    y = torch.empty(M, N, dtype=torch.float32, device=x.device)
    rc = lib.loopspec_op_linear(W.data_ptr(), 1 if W.dtype == torch.bfloat16 else 0, x.data_ptr(), y.data_ptr(), M, N, K,
                                scratch.data_ptr(), scratch.numel(), torch.cuda.current_stream().cuda_stream)
    if rc:
        raise LoopSpecError(rc)
    return y


def linear_tc(W, x, scratch=None, check=True):
    """y = x @ W.T through the tcgen05 / TMA operator.  W [N,K] bf16 (read in place), x [M,K] fp32 (cuda tensors).
    check: synchronise and raise if a bounded wait inside the kernel ran out."""
    import torch
    M, K = x.shape
    N = W.shape[0]
    need = lib.loopspec_linear_tc_scratch_bytes(M, N, K)
    if need == 0 or W.dtype != torch.bfloat16:
        raise LoopSpecError(-1, "unsupported linear_tc shape or dtype")
    if scratch is None:
        scratch = torch.empty(need + 256, dtype=torch.uint8, device=x.device)
    off = (-scratch.data_ptr()) % 256
    y = torch.empty(M, N, dtype=torch.float32, device=x.device)
    rc = lib.loopspec_op_linear_tc(W.data_ptr(), x.data_ptr(), y.data_ptr(), M, N, K, scratch.data_ptr() + off,
                                   scratch.numel() - off, torch.cuda.current_stream().cuda_stream)
    if rc:
        raise LoopSpecError(rc, "op_linear_tc")
    if check:
        torch.cuda.current_stream().synchronize()
        if int(scratch[off:off + 4].view(torch.int32).item()) != 0:
            raise LoopSpecError(-5, "op_linear_tc: a bounded device-side wait ran out")
    return y


def time_linear_tc(Ws, x, iters=10):
    """Mean microseconds per launch of the tcgen05 kernel alone, back to back over the weight matrices Ws."""
    import torch
    M, K = x.shape
    N = Ws[0].shape[0]
    need = lib.loopspec_linear_tc_scratch_bytes(M, N, K)
    if need == 0:
        raise LoopSpecError(-1, "unsupported linear_tc shape")
    scratch = torch.empty(need + 256, dtype=torch.uint8, device=x.device)
    off = (-scratch.data_ptr()) % 256
    ptrs = (C.c_void_p * len(Ws))(*[w.data_ptr() for w in Ws])
    us = C.c_float(0)
    rc = lib.loopspec_time_linear_tc(ptrs, len(Ws), x.data_ptr(), M, N, K, scratch.data_ptr() + off, scratch.numel() - off,
                                     iters, C.byref(us), torch.cuda.current_stream().cuda_stream)
    if rc:
        raise LoopSpecError(rc, "time_linear_tc")
    if int(scratch[off:off + 4].view(torch.int32).item()) != 0:
        raise LoopSpecError(-5, "time_linear_tc: a bounded device-side wait ran out")
    return us.value


def linear_static(W, x):
    """y = x @ W.T like `linear`, but through the entry point that needs no scratch buffer from the caller: for
    processes that may not allocate device memory while serving.  Only the output tensor is created here."""
    import torch
    M, K = x.shape
    N = W.shape[0]
    y = torch.empty(M, N, dtype=torch.float32, device=x.device)
    rc = lib.loopspec_op_linear_static(W.data_ptr(), 1 if W.dtype == torch.bfloat16 else 0, x.data_ptr(), y.data_ptr(), M, N, K,
                                       torch.cuda.current_stream().cuda_stream)
    if rc:
        raise LoopSpecError(rc, "op_linear_static")
    return y


class LoopSpec:
    """One decoding context (see include/loopspec.h for the semantics of every call)."""

    def __init__(self, shape, weights, d1=1, d2=0, temperature=0.0, seed=0, gate=True, residual_q2=True, max_seqs=1,
                 max_ctx=2048, alpha=0.0, beta=0.0, max_prefill_rows=0, stream=None, top_k=0, top_p=1.0, measure_tv=False, mask_first=False, prefill_skinny=False):
        import torch
        self._torch = torch
        self.shape = shape
        self.h = None
        self.weights = weights  # keep the tensors alive: the library borrows them
        # CUDA graphs cannot be captured on the legacy default stream: the context gets a stream of its own
        self.stream = stream or torch.cuda.Stream()
        torch.cuda.synchronize()  # weights were uploaded on other streams
        self.model = Model(shape.vocab, shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn,
                           shape.n_prelude, shape.n_recurrent, shape.n_coda, shape.R,
                           1 if shape.weight_dtype == "bf16" else 0, 1 if shape.tied else 0, shape.rms_eps, shape.rope_theta)
        self.sched = Sched(d1, d2, alpha, beta, int(gate), int(residual_q2), temperature, seed, max_seqs, max_ctx,
                           max_prefill_rows, int(top_k), float(top_p), int(measure_tv), int(mask_first), int(prefill_skinny))
        nbytes = lib.loopspec_workspace_bytes(C.byref(self.model), C.byref(self.sched))
        if nbytes == 0:
            # let init report the precise status
            nbytes = 256
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        names = ["norm1", "wqkv", "wo", "norm2", "wgateup", "wdown"]
        blocks = [(f"prelude.{l}") for l in range(shape.n_prelude)] + [f"layers.{l}" for l in range(shape.n_recurrent)] + \
                 [f"coda.{l}" for l in range(shape.n_coda)]
        ptrs = (C.c_void_p * (6 * len(blocks)))()
        for i, blk in enumerate(blocks):
            for j, n in enumerate(names):
                ptrs[6 * i + j] = weights[f"{blk}.{n}"].data_ptr()
        self._ptrs = ptrs
        adapter = weights["adapter"].data_ptr() if (shape.n_prelude or shape.n_coda) else None
        wt = Weights(weights["embed"].data_ptr(), 0 if shape.tied else weights["lm_head"].data_ptr(),
                     weights["final_norm"].data_ptr(), adapter, C.cast(ptrs, C.POINTER(C.c_void_p)))
        h = C.c_void_p()
        rc = lib.loopspec_init(C.byref(self.model), C.byref(self.sched), C.byref(wt), self.workspace.data_ptr(), nbytes,
                               self.stream.cuda_stream, C.byref(h))
        if rc:
            raise LoopSpecError(rc, "init")
        self.h = h
        self.max_seqs = max_seqs
        self.workspace_bytes = nbytes

    def _check(self, rc):
        if rc:
            raise LoopSpecError(rc, lib.loopspec_last_error(self.h).decode())

    def close(self):
        if self.h is not None:
            lib.loopspec_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def prefill(self, prompt, seq=0):
        ids = np.ascontiguousarray(prompt, dtype=np.int32)
        first = C.c_int32()
        self._check(lib.loopspec_prefill(self.h, seq, ids.ctypes.data_as(C.POINTER(C.c_int32)), len(ids), C.byref(first)))
        return first.value

    def step(self):
        a, b = C.c_int32(), C.c_int32()
        self._check(lib.loopspec_step(self.h, C.byref(a), C.byref(b)))
        return a.value, b.value

    @staticmethod
    def _commit_dict(c):
        return {n: getattr(c, n) for n, _ in Commit._fields_}

    def verify(self):
        out = (Commit * self.max_seqs)()
        n = C.c_int32()
        self._check(lib.loopspec_verify(self.h, out, self.max_seqs, C.byref(n)))
        return [self._commit_dict(out[i]) for i in range(min(n.value, self.max_seqs))]

    def _decode(self, fn, n):
        out = np.full((self.max_seqs, n), -1, dtype=np.int32)
        self._check(fn(self.h, n, out.ctypes.data_as(C.POINTER(C.c_int32))))
        return out

    def decode(self, n):
        return self._decode(lib.loopspec_decode, n)

    def vanilla_decode(self, n):
        return self._decode(lib.loopspec_vanilla_decode, n)

    def debug_drop_tile(self, unit, wait_us=100):
        self._check(lib.loopspec_debug_drop_tile(self.h, unit, wait_us))

    def stats(self):
        s = Stats()
        self._check(lib.loopspec_get_stats(self.h, C.byref(s)))
        return {n: getattr(s, n) for n, _ in Stats._fields_}

    def commits(self, seq=0):
        n = C.c_int32()
        self._check(lib.loopspec_get_commits(self.h, seq, None, 0, C.byref(n)))
        out = (Commit * max(n.value, 1))()
        self._check(lib.loopspec_get_commits(self.h, seq, out, n.value, C.byref(n)))
        return [self._commit_dict(out[i]) for i in range(n.value)]

    def row_trace(self):
        n = C.c_int32()
        self._check(lib.loopspec_get_row_trace(self.h, None, 0, C.byref(n)))
        out = np.zeros(max(n.value, 1), dtype=np.int32)
        self._check(lib.loopspec_get_row_trace(self.h, out.ctypes.data_as(C.POINTER(C.c_int32)), n.value, C.byref(n)))
        return out[: n.value]

    def debug_logits(self, seq=0, which=0):
        out = np.zeros(self.shape.vocab, dtype=np.float32)
        self._check(lib.loopspec_debug_logits(self.h, seq, which, out.ctypes.data_as(C.POINTER(C.c_float))))
        return out

    def launches_per_step(self):
        n = C.c_int32()
        self._check(lib.loopspec_launches_per_step(self.h, C.byref(n)))
        return n.value

    def decode_paths(self):
        """(gemm_path, attention_path) of this context's decode passes: see loopspec_decode_paths."""
        g, a = C.c_int32(), C.c_int32()
        self._check(lib.loopspec_decode_paths(self.h, C.byref(g), C.byref(a)))
        return g.value, a.value

    def time_kernel(self, which, rows, iters):
        ms, nbytes = C.c_float(), C.c_double()
        self._check(lib.loopspec_time_kernel(self.h, which, rows, iters, C.byref(ms), C.byref(nbytes)))
        return ms.value, nbytes.value
