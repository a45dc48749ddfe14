"""ctypes binding of libil.so: argument marshalling only — every step of the training path runs in
the CUDA library.  torch is used for device memory (allocator hook), CUDA streams and host/device
tensors handed to the operator-level calls."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libil.so")

IL_OK = 0
STATUS = {0: "IL_OK", 1: "IL_ERR_INVALID_ARG", 2: "IL_ERR_STATE", 3: "IL_ERR_OOM", 4: "IL_ERR_CUDA",
          5: "IL_ERR_TIMEOUT", 6: "IL_ERR_NONFINITE"}


class ILError(RuntimeError):
    def __init__(self, status: int, msg: str = ""):
        self.status = status
        super().__init__(f"{STATUS.get(status, status)}: {msg}")


ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_size_t, C.c_void_p)
FREE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)


class il_options(C.Structure):
    _fields_ = [("device", C.c_int), ("max_batch", C.c_int), ("max_seq", C.c_int),
                ("alloc", ALLOC_FN), ("free_", FREE_FN), ("alloc_ctx", C.c_void_p),
                ("streams", C.POINTER(C.c_void_p)), ("n_streams", C.c_int),
                ("use_bias", C.c_int), ("ln_eps", C.c_float), ("head_layers", C.c_int),
                ("head_mode", C.c_int), ("placement", C.c_int), ("attn_bwd", C.c_int),
                ("devices", C.POINTER(C.c_int)), ("n_devices", C.c_int)]


class il_gemm_desc(C.Structure):
    _fields_ = [("M", C.c_int), ("N", C.c_int), ("K", C.c_int),
                ("A", C.c_void_p), ("lda", C.c_int), ("a_mn_major", C.c_int),
                ("B", C.c_void_p), ("ldb", C.c_int), ("b_mn_major", C.c_int),
                ("epilogue", C.c_int),
                ("C", C.c_void_p), ("ldc", C.c_int),
                ("C2", C.c_void_p),
                ("bias", C.c_void_p), ("resid", C.c_void_p),
                ("aux", C.c_void_p), ("ld_aux", C.c_int), ("aux_rows", C.c_int), ("colsum", C.c_void_p),
                ("accumulate", C.c_int), ("split_k", C.c_int),
                ("targets", C.c_void_p),
                ("part_max", C.c_void_p), ("part_sum", C.c_void_p), ("part_ld", C.c_int),
                ("tgt_logit", C.c_void_p), ("lse", C.c_void_p),
                ("scale", C.c_float), ("col0", C.c_int), ("tile_blocks", C.c_int),
                ("rowscale", C.c_void_p), ("store_exp", C.c_int)]


_lib = None


def lib() -> C.CDLL:
    """Load libil.so (built in-tree by paper_2010_04116_b200.build); fails loudly when it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2010_04116_b200.build` "
                          "(there is no fallback path)")
    L = C.CDLL(LIB_PATH)
    vp, i, f, sz = C.c_void_p, C.c_int, C.c_float, C.c_size_t
    sig = {
        "il_create": [i, i, i, i, i, i, i, C.POINTER(il_options), C.POINTER(vp)],
        "il_destroy": [vp], "il_set_n": [vp, i], "il_set_rule": [vp, i], "il_set_micro_batches": [vp, i],
        "il_lr_schedule": [C.c_longlong, i, i, C.POINTER(C.c_double)],
        "il_tensor_info": [vp, i, C.POINTER(C.c_char_p), C.POINTER(i), C.POINTER(i), C.POINTER(i),
                           C.POINTER(C.c_longlong)],
        "il_set_param": [vp, i, vp, sz], "il_get_param": [vp, i, vp, sz], "il_get_grad": [vp, i, vp, sz],
        "il_get_opt_state": [vp, i, vp, vp, C.POINTER(C.c_longlong)],
        "il_set_opt_state": [vp, i, vp, vp, C.c_longlong],
        "il_set_batch": [vp, vp, vp, i, i, i],
        "il_forward_component": [vp, i], "il_aux_head_loss": [vp, i, C.POINTER(f)],
        "il_get_losses": [vp, C.POINTER(f)], "il_backward_nwise": [vp],
        "il_adamw_step": [vp, f, f, f, f, f], "il_sync": [vp],
        "il_get_boundary": [vp, i, vp, sz],
        "il_get_token_losses": [vp, i, vp, sz],
        "il_stats": [vp, C.POINTER(C.c_longlong), C.POINTER(C.c_longlong)],
        "il_profile": [vp, i],
        "il_profile_read": [vp, C.POINTER(C.c_double), C.POINTER(C.c_longlong), C.POINTER(C.c_double)],
        "il_nwise_streams": [i, i, i, C.POINTER(i), C.POINTER(i)],
        "il_pipeline_transfers": [i, i, i, C.POINTER(i), i, C.POINTER(i)],
        "il_pipeline_last_transfers": [vp, C.POINTER(i), i, C.POINTER(i)],
        "il_error_word": [vp, i, C.POINTER(vp)],
        "il_head_mode": [vp],
        "il_op_wait_probe": [vp, C.c_uint, vp],
        "il_op_attention_bwd_noalloc_status": [vp],
        "il_time_per_batch": [i, i, i, C.c_double, C.c_double, C.POINTER(C.c_double)],
        "il_optimal_microbatches": [i, i, C.c_double, C.c_double, i, C.POINTER(i)],
        "il_op_gemm": [C.POINTER(il_gemm_desc), vp, vp],
        "il_op_attention_fwd": [vp, vp, vp, i, i, i, i, vp],
        "il_op_attention_bwd": [vp, vp, vp, vp, vp, vp, i, i, i, i, i, vp],
        "il_op_attention_bwd_noalloc": [vp, vp, vp, vp, vp, i, i, i, i, i, vp],
        "il_op_attention_bwd_one_sweep": [vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, vp, vp],
        "il_op_layernorm_fwd": [vp, vp, vp, vp, vp, vp, i, i, f, vp],
        "il_op_layernorm_bwd": [vp, i, vp, vp, vp, vp, vp, vp, vp, vp, vp, i, i, i, vp],
        "il_op_layernorm_bwd_fused": [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i, i, i, vp],
    }
    for name, args in sig.items():
        fn = getattr(L, name)
        fn.argtypes = args
        fn.restype = C.c_int
    L.il_op_attention_bwd_noalloc_max_rows.argtypes = []
    L.il_op_attention_bwd_noalloc_max_rows.restype = C.c_size_t
    L.il_num_tensors.argtypes = [vp]
    L.il_num_tensors.restype = C.c_int
    L.il_last_error.argtypes = [vp]
    L.il_last_error.restype = C.c_char_p
    L.il_status_string.argtypes = [C.c_int]
    L.il_status_string.restype = C.c_char_p
    _lib = L
    return L


def nwise_streams(K: int, n: int, k: int) -> List[int]:
    terms = (C.c_int * max(K, 1))()
    cnt = C.c_int(0)
    st = lib().il_nwise_streams(K, n, k, terms, C.byref(cnt))
    if st != IL_OK:
        raise ILError(st, "il_nwise_streams")
    return [terms[i] for i in range(cnt.value)]


RULES = {"sum": 0, "far": 1, "mean": 2}


def pipeline_transfers(K: int, n: int, rule: str = "sum") -> List[tuple]:
    """(direction, boundary, id) of every tensor that crosses a component boundary in one step of the pipeline
    placement, in issue order (host-only)."""
    cnt = C.c_int(0)
    st = lib().il_pipeline_transfers(K, n, RULES[rule], None, 0, C.byref(cnt))
    if st != IL_OK:
        raise ILError(st, "il_pipeline_transfers")
    rec = (C.c_int * (3 * max(cnt.value, 1)))()
    st = lib().il_pipeline_transfers(K, n, RULES[rule], rec, cnt.value, C.byref(cnt))
    if st != IL_OK:
        raise ILError(st, "il_pipeline_transfers")
    return [(rec[3 * i], rec[3 * i + 1], rec[3 * i + 2]) for i in range(cnt.value)]


def time_per_batch(A: int, M: int, N: int, c0: float, c1: float) -> float:
    out = C.c_double(0)
    st = lib().il_time_per_batch(A, M, N, c0, c1, C.byref(out))
    if st != IL_OK:
        raise ILError(st, "il_time_per_batch")
    return out.value


def lr_schedule(step: int, d_model: int, warmup_steps: int = 4000) -> float:
    out = C.c_double(0)
    st = lib().il_lr_schedule(step, d_model, warmup_steps, C.byref(out))
    if st != IL_OK:
        raise ILError(st, "il_lr_schedule")
    return out.value


def optimal_microbatches(A: int, N: int, c0: float, c1: float, max_log2: int = 10) -> int:
    out = C.c_int(0)
    st = lib().il_optimal_microbatches(A, N, c0, c1, max_log2, C.byref(out))
    if st != IL_OK:
        raise ILError(st, "il_optimal_microbatches")
    return out.value


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    return t.data_ptr()


class Model:
    """One il_model.  Device memory comes from torch's caching allocator through the allocator hook and
    the K per-component streams are torch streams."""

    def __init__(self, K: int, Lc: int, d: int, H: int, F: int, V: int, n: int, max_batch: int, max_seq: int,
                 device: int = 0, torch_alloc: bool = True, torch_streams: bool = True, head_layers: int = 0,
                 head_mode: str = "stored", placement: str = "single", devices: Optional[Sequence[int]] = None,
                 alloc_fail_at: Optional[int] = None, attn_bwd: str = "one_sweep"):
        """head_mode: 'stored' (exp(logits) kept for the backward) or 'recompute' (vocabulary-chunked backward that
        forms the logits again).  placement: 'single', or 'pipeline' = one component per entry of `devices`
        (default: all on `device`, still exchanged through the copy path).  alloc_fail_at: make the allocator
        hook return NULL at its i-th call (0-based), for tests of the out-of-memory path."""
        import torch
        self._torch = torch
        self.L = lib()
        self.K, self.Lc, self.d, self.H, self.F, self.V, self.n = K, Lc, d, H, F, V, n
        self.device = device
        self._blocks: Dict[int, object] = {}
        self._h = C.c_void_p(None)
        opt = il_options()
        opt.device = device
        opt.max_batch, opt.max_seq = max_batch, max_seq
        opt.use_bias = 1
        opt.ln_eps = 1e-5
        opt.head_layers = head_layers
        opt.head_mode = {"stored": 0, "recompute": 1}[head_mode]
        opt.placement = {"single": 0, "pipeline": 1}[placement]
        opt.attn_bwd = {"one_sweep": 0, "two_kernels": 1}[attn_bwd]
        self.placement = placement
        self.devices = list(devices) if devices is not None else [device] * K
        if devices is not None:
            self._dev_arr = (C.c_int * K)(*self.devices)
            opt.devices = C.cast(self._dev_arr, C.POINTER(C.c_int))
            opt.n_devices = K
        dev = torch.device("cuda", device)
        self._alloc_calls = 0
        if torch_alloc:
            def _alloc(nbytes, ctx):
                i = self._alloc_calls
                self._alloc_calls += 1
                if alloc_fail_at is not None and i == alloc_fail_at:
                    return None
                try:
                    # the library calls the hook with the target device current
                    cur = torch.device("cuda", torch.cuda.current_device()) if devices is not None else dev
                    t = torch.empty(int(nbytes), dtype=torch.uint8, device=cur)
                except Exception:
                    return None
                self._blocks[t.data_ptr()] = t
                return t.data_ptr()

            def _free(p, ctx):
                self._blocks.pop(p, None)

            self._alloc_cb, self._free_cb = ALLOC_FN(_alloc), FREE_FN(_free)
            opt.alloc, opt.free_ = self._alloc_cb, self._free_cb
        self.streams = []
        if torch_streams:
            self.streams = [torch.cuda.Stream(device=torch.device("cuda", self.devices[k])) for k in range(K)]
            self._stream_arr = (C.c_void_p * K)(*[s.cuda_stream for s in self.streams])
            opt.streams = C.cast(self._stream_arr, C.POINTER(C.c_void_p))
            opt.n_streams = K
        self._opt = opt
        st = self.L.il_create(K, Lc, d, H, F, V, n, C.byref(opt), C.byref(self._h))
        if st != IL_OK:
            msg = self.L.il_last_error(self._h).decode() if self._h else ""
            if self._h:
                self.L.il_destroy(self._h)
                self._h = C.c_void_p(None)
            raise ILError(st, msg)
        self.names: List[str] = []
        self.shapes: Dict[str, tuple] = {}
        self.index: Dict[str, int] = {}
        for i in range(self.L.il_num_tensors(self._h)):
            name = C.c_char_p()
            comp, is_head, rank = C.c_int(), C.c_int(), C.c_int()
            shape = (C.c_longlong * 2)()
            self._ck(self.L.il_tensor_info(self._h, i, C.byref(name), C.byref(comp), C.byref(is_head),
                                           C.byref(rank), shape))
            nm = name.value.decode()
            self.names.append(nm)
            self.index[nm] = i
            self.shapes[nm] = (int(shape[0]), int(shape[1])) if rank.value == 2 else (int(shape[0]),)

    # ------------------------------------------------------------------ plumbing
    def _ck(self, st: int):
        if st != IL_OK:
            raise ILError(st, self.L.il_last_error(self._h).decode())

    def close(self):
        if self._h:
            self.L.il_destroy(self._h)
            self._h = C.c_void_p(None)
            self._blocks.clear()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ parameters
    def set_param(self, name: str, value: np.ndarray):
        v = np.ascontiguousarray(value, dtype=np.float32)
        self._ck(self.L.il_set_param(self._h, self.index[name], v.ctypes.data, v.size))

    def set_params(self, params: Dict[str, np.ndarray]):
        for k, v in params.items():
            self.set_param(k, v)

    def _get(self, fn, name: str) -> np.ndarray:
        out = np.empty(self.shapes[name], dtype=np.float32)
        self._ck(fn(self._h, self.index[name], out.ctypes.data, out.size))
        return out

    def get_param(self, name: str) -> np.ndarray:
        return self._get(self.L.il_get_param, name)

    def get_grad(self, name: str) -> np.ndarray:
        return self._get(self.L.il_get_grad, name)

    def get_opt_state(self, name: str):
        m = np.empty(self.shapes[name], dtype=np.float32)
        v = np.empty(self.shapes[name], dtype=np.float32)
        step = C.c_longlong(0)
        self._ck(self.L.il_get_opt_state(self._h, self.index[name], m.ctypes.data, v.ctypes.data, C.byref(step)))
        return m, v, step.value

    def set_opt_state(self, name: str, m: np.ndarray, v: np.ndarray, step: int):
        m = np.ascontiguousarray(m, dtype=np.float32)
        v = np.ascontiguousarray(v, dtype=np.float32)
        self._ck(self.L.il_set_opt_state(self._h, self.index[name], m.ctypes.data, v.ctypes.data, step))

    RULES = RULES

    def error_word(self, k: int = 0) -> int:
        """Device address of the error word component k's kernels report to."""
        out = C.c_void_p(None)
        self._ck(self.L.il_error_word(self._h, k, C.byref(out)))
        return out.value

    def last_transfers(self) -> List[tuple]:
        """(direction, boundary, id) of the copies between components issued since the last set_batch."""
        cnt = C.c_int(0)
        self._ck(self.L.il_pipeline_last_transfers(self._h, None, 0, C.byref(cnt)))
        rec = (C.c_int * (3 * max(cnt.value, 1)))()
        self._ck(self.L.il_pipeline_last_transfers(self._h, rec, cnt.value, C.byref(cnt)))
        return [(rec[3 * i], rec[3 * i + 1], rec[3 * i + 2]) for i in range(cnt.value)]

    def set_rule(self, rule: str):
        """'sum' (default), 'far' (the paper's main-text rule) or 'mean' (its Transformer variant)."""
        self._ck(self.L.il_set_rule(self._h, self.RULES[rule]))

    def set_micro_batches(self, micro_batches: int):
        """Process every mini-batch as this many micro-batch steps before one update (Sec. 3.1)."""
        self._ck(self.L.il_set_micro_batches(self._h, micro_batches))

    def set_n(self, n: int):
        self._ck(self.L.il_set_n(self._h, n))
        self.n = n

    # ------------------------------------------------------------------ the step
    def set_batch(self, tokens, targets):
        """tokens/targets [B, T] int32: numpy arrays / CPU tensors (host) or CUDA tensors (device)."""
        torch = self._torch
        if isinstance(tokens, np.ndarray):
            tokens = np.ascontiguousarray(tokens, dtype=np.int32)
            targets = np.ascontiguousarray(targets, dtype=np.int32)
            B, T = tokens.shape
            self._keep = (tokens, targets)
            self._ck(self.L.il_set_batch(self._h, tokens.ctypes.data, targets.ctypes.data, B, T, 0))
        else:
            assert tokens.dtype == torch.int32 and targets.dtype == torch.int32
            tokens, targets = tokens.contiguous(), targets.contiguous()
            B, T = tokens.shape
            self._keep = (tokens, targets)
            self._ck(self.L.il_set_batch(self._h, tokens.data_ptr(), targets.data_ptr(), B, T,
                                         1 if tokens.is_cuda else 0))

    def forward_component(self, k: int):
        self._ck(self.L.il_forward_component(self._h, k))

    def aux_head_loss(self, k: int, sync: bool = False) -> Optional[float]:
        if sync:
            out = C.c_float(0)
            self._ck(self.L.il_aux_head_loss(self._h, k, C.byref(out)))
            return out.value
        self._ck(self.L.il_aux_head_loss(self._h, k, None))
        return None

    def get_losses(self) -> np.ndarray:
        out = (C.c_float * self.K)()
        self._ck(self.L.il_get_losses(self._h, out))
        return np.array(list(out), dtype=np.float32)

    def get_token_losses(self, k: int, ntok: int) -> np.ndarray:
        out = np.empty(ntok, dtype=np.float32)
        self._ck(self.L.il_get_token_losses(self._h, k, out.ctypes.data, out.size))
        return out

    def backward_nwise(self):
        self._ck(self.L.il_backward_nwise(self._h))

    def adamw_step(self, lr: float, beta1: float = 0.9, beta2: float = 0.98, eps: float = 1e-9,
                   weight_decay: float = 0.0):
        self._ck(self.L.il_adamw_step(self._h, lr, beta1, beta2, eps, weight_decay))

    def sync(self):
        self._ck(self.L.il_sync(self._h))

    def get_boundary(self, k: int, ntok: int) -> np.ndarray:
        out = np.empty((ntok, self.d), dtype=np.float32)
        self._ck(self.L.il_get_boundary(self._h, k, out.ctypes.data, out.size))
        return out

    @property
    def head_mode(self) -> str:
        """The head mode in force: a stored-mode model switches to "recompute" when a row leaves the stored form's range."""
        return {0: "stored", 1: "recompute"}[self.L.il_head_mode(self._h)]

    def stats(self):
        b, l = C.c_longlong(0), C.c_longlong(0)
        self._ck(self.L.il_stats(self._h, C.byref(b), C.byref(l)))
        return b.value, l.value

    def profile(self, enable):
        """0/False off, 1/True events around each GEMM, 2 the same with each GEMM alone on the GPU."""
        self._ck(self.L.il_profile(self._h, int(enable)))

    def profile_read(self):
        ms, n, fl = C.c_double(0), C.c_longlong(0), C.c_double(0)
        self._ck(self.L.il_profile_read(self._h, C.byref(ms), C.byref(n), C.byref(fl)))
        return ms.value, n.value, fl.value

    def train_step(self, tokens, targets, adamw: Optional[dict] = None):
        """set_batch -> K forwards with their heads -> n-wise backward (-> AdamW).  Asynchronous."""
        self.set_batch(tokens, targets)
        for k in range(self.K):
            self.forward_component(k)
            self.aux_head_loss(k)
        self.backward_nwise()
        if adamw is not None:
            self.adamw_step(**adamw)

    def train_minibatch(self, tokens, targets, micro_batches: int, adamw: Optional[dict] = None):
        """One update from a mini-batch processed as `micro_batches` equal groups of sequences (Sec. 3.1);
        il_set_micro_batches(micro_batches) must be in effect.  Asynchronous."""
        per = tokens.shape[0] // micro_batches
        for mb in range(micro_batches):
            self.train_step(tokens[mb * per:(mb + 1) * per], targets[mb * per:(mb + 1) * per])
        if adamw is not None:
            self.adamw_step(**adamw)


# ---------------------------------------------------------------------- operator-level calls
def op_gemm(M, N, K, A, lda, a_mn, B, ldb, b_mn, epilogue, err_word, C_=None, ldc=0, C2=None, bias=None,
            resid=None, aux=None, ld_aux=0, aux_rows=0, colsum=None, accumulate=0, split_k=0, targets=None, part_max=None,
            part_sum=None, part_ld=0, tgt_logit=None, lse=None, scale=0.0, col0=0, tile_blocks=0, rowscale=None, store_exp=0, stream=None):
    d = il_gemm_desc()
    d.M, d.N, d.K = M, N, K
    d.A, d.lda, d.a_mn_major = _ptr(A), lda, a_mn
    d.B, d.ldb, d.b_mn_major = _ptr(B), ldb, b_mn
    d.epilogue = epilogue
    d.C, d.ldc, d.C2 = _ptr(C_), ldc, _ptr(C2)
    d.bias, d.resid = _ptr(bias), _ptr(resid)
    d.aux, d.ld_aux, d.aux_rows = _ptr(aux), ld_aux, aux_rows
    d.colsum = _ptr(colsum)
    d.accumulate = accumulate
    d.split_k = split_k
    d.targets = _ptr(targets)
    d.part_max, d.part_sum, d.part_ld = _ptr(part_max), _ptr(part_sum), part_ld
    d.tgt_logit, d.lse = _ptr(tgt_logit), _ptr(lse)
    d.scale, d.col0 = scale, col0
    d.tile_blocks = tile_blocks
    d.rowscale, d.store_exp = _ptr(rowscale), store_exp
    st = lib().il_op_gemm(C.byref(d), _ptr(err_word), stream)
    if st != IL_OK:
        raise ILError(st, "il_op_gemm")


def op_attention_fwd(qkv, o, lse, B, T, H, dh, stream=None):
    st = lib().il_op_attention_fwd(_ptr(qkv), _ptr(o), _ptr(lse), B, T, H, dh, stream)
    if st != IL_OK:
        raise ILError(st, "il_op_attention_fwd")


def op_attention_bwd(qkv, o, lse, dout, dqkv, delta, NB, B, T, H, dh, stream=None):
    st = lib().il_op_attention_bwd(_ptr(qkv), _ptr(o), _ptr(lse), _ptr(dout), _ptr(dqkv), _ptr(delta), NB, B, T, H,
                                   dh, stream)
    if st != IL_OK:
        raise ILError(st, "il_op_attention_bwd")


def op_attention_bwd_one_sweep(qkv, o, lse, dout, dqkv, delta, dq_acc, NB, B, T, H, dh, err_word=None, stream=None):
    st = lib().il_op_attention_bwd_one_sweep(_ptr(qkv), _ptr(o), _ptr(lse), _ptr(dout), _ptr(dqkv), _ptr(delta),
                                             _ptr(dq_acc), NB, B, T, H, dh, _ptr(err_word), stream)
    if st != IL_OK:
        raise ILError(st, "il_op_attention_bwd_one_sweep")


def op_wait_probe(err_word_ptr: int, limit_us: int, stream=None):
    """Launch the error-path probe: a bounded wait that runs out after limit_us and writes a time-out code to the
    device word at err_word_ptr."""
    st = lib().il_op_wait_probe(err_word_ptr, limit_us, stream)
    if st != IL_OK:
        raise ILError(st, "il_op_wait_probe")


def op_attention_bwd_noalloc_status(stream=None) -> int:
    """il_status of the allocation-free attention backward calls since the last query (0 = fine)."""
    return lib().il_op_attention_bwd_noalloc_status(stream)


def op_attention_bwd_noalloc(qkv, o, lse, dout, dqkv, NB, B, T, H, dh, stream=None):
    """Attention backward whose scratch is a fixed array inside the library: allocates nothing."""
    st = lib().il_op_attention_bwd_noalloc(_ptr(qkv), _ptr(o), _ptr(lse), _ptr(dout), _ptr(dqkv), NB, B, T, H, dh,
                                           stream)
    if st != IL_OK:
        raise ILError(st, "il_op_attention_bwd_noalloc")


def op_layernorm_fwd(x, gamma, beta, y, mean, rstd, rows, d, eps=1e-5, stream=None):
    st = lib().il_op_layernorm_fwd(_ptr(x), _ptr(gamma), _ptr(beta), _ptr(y), _ptr(mean), _ptr(rstd), rows, d, eps,
                                   stream)
    if st != IL_OK:
        raise ILError(st, "il_op_layernorm_fwd")


def op_layernorm_bwd(dy, dy_is_f32, x, mean, rstd, gamma, resid, dx, dx_bf16, dgamma, dbeta, rows, x_rows, d,
                     stream=None):
    st = lib().il_op_layernorm_bwd(_ptr(dy), dy_is_f32, _ptr(x), _ptr(mean), _ptr(rstd), _ptr(gamma), _ptr(resid),
                                   _ptr(dx), _ptr(dx_bf16), _ptr(dgamma), _ptr(dbeta), rows, x_rows, d, stream)
    if st != IL_OK:
        raise ILError(st, "il_op_layernorm_bwd")


def op_layernorm_bwd_fused(dy, x, mean, rstd, gamma, resid, dx, dx_bf16, dgamma, dbeta, colsum, rows, x_rows, d,
                           stream=None):
    st = lib().il_op_layernorm_bwd_fused(_ptr(dy), _ptr(x), _ptr(mean), _ptr(rstd), _ptr(gamma), _ptr(resid), _ptr(dx),
                                         _ptr(dx_bf16), _ptr(dgamma), _ptr(dbeta), _ptr(colsum), rows, x_rows, d, stream)
    if st != IL_OK:
        raise ILError(st, "il_op_layernorm_bwd_fused")
