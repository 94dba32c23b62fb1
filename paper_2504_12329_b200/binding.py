"""ctypes binding of libst.so: the same entry points as include/st.h, argument marshalling only.

Device memory handed to the library (and, optionally, the library's own weights and KV pools through
the allocator hooks) comes from PyTorch; every computation runs in the library's CUDA kernels.  If
the shared library is missing the import fails -- there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libst.so")

ST_OK, ST_ERR_ARG, ST_ERR_OOM, ST_ERR_KV_FULL, ST_ERR_VOCAB = 0, -1, -2, -3, -4
ST_ERR_TIMEOUT, ST_ERR_UNSUPPORTED, ST_ERR_INTERNAL, ST_ERR_CAPACITY = -5, -6, -7, -8

ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_uint64, C.c_void_p)
FREE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)


class StConfig(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("hidden", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("ffn", C.c_int32), ("vocab", C.c_int32),
        ("rope_theta", C.c_float), ("rms_eps", C.c_float),
        ("tie_embeddings", C.c_int32), ("qkv_bias", C.c_int32),
        ("max_seqs", C.c_int32), ("max_tokens", C.c_int32), ("page_size", C.c_int32),
        ("alloc", ALLOC_FN), ("free", FREE_FN), ("alloc_user", C.c_void_p),
    ]


class StSpecParams(C.Structure):
    _fields_ = [
        ("delimiter_id", C.c_int32), ("keyword_ids", C.POINTER(C.c_int32)), ("n_keywords", C.c_int32),
        ("n1", C.c_int32), ("keep_probe", C.c_int32), ("eos_id", C.c_int32), ("vocab_limit", C.c_int32),
        ("max_new_tokens", C.c_int32), ("takeover_every_delimiter", C.c_int32), ("target_first_n", C.c_int32),
        ("affirmation_ids", C.POINTER(C.c_int32)), ("n_affirmation", C.c_int32),
        ("verification_ids", C.POINTER(C.c_int32)), ("n_verification", C.c_int32),
        ("n2", C.c_int32), ("neg_threshold", C.c_int32), ("n3", C.c_int32),
        ("aux_ids", C.POINTER(C.c_int32)), ("n_aux", C.c_int32), ("probe_len", C.c_int32),
        ("delimiter_ids", C.POINTER(C.c_int32)), ("n_delimiters", C.c_int32),
        ("temperature", C.c_float), ("sample_seed", C.c_uint64), ("top_p", C.c_float),
    ]


class StHandoff(C.Structure):
    _fields_ = [("seg_start", C.c_int32), ("step", C.c_int32), ("catchup_len", C.c_int32)]


class StSpecResult(C.Structure):
    _fields_ = [
        ("tokens", C.POINTER(C.c_int32)), ("source", C.POINTER(C.c_uint8)),
        ("cap_tokens", C.c_int32), ("n_tokens", C.c_int32),
        ("handoffs", C.POINTER(StHandoff)), ("cap_handoffs", C.c_int32), ("n_handoffs", C.c_int32),
        ("emission_tokens", C.POINTER(C.c_int32)), ("emission_source", C.POINTER(C.c_uint8)),
        ("emission_fed", C.POINTER(C.c_int32)), ("emission_argmax", C.POINTER(C.c_int32)),
        ("cap_steps", C.c_int32), ("n_steps", C.c_int32),
        ("kv_len_small", C.c_int32), ("kv_len_large", C.c_int32),
        ("logits_trace", C.POINTER(C.c_float)), ("trace_first_step", C.c_int32), ("trace_n_steps", C.c_int32),
        ("seconds", C.c_double), ("bytes_algorithmic", C.c_int64),
        ("handoff_kinds", C.POINTER(C.c_uint8)),
        ("t_prompt_prefill_s", C.c_double), ("t_catchup_s", C.c_double), ("t_decode_s", C.c_double),
        ("n_prompt_prefill", C.c_int32), ("n_catchup", C.c_int32), ("n_decode", C.c_int32),
    ]


class StSpecDecParams(C.Structure):
    _fields_ = [("gamma", C.c_int32), ("eos_id", C.c_int32), ("vocab_limit", C.c_int32), ("max_new_tokens", C.c_int32)]


class StSpecDecResult(C.Structure):
    _fields_ = [
        ("tokens", C.POINTER(C.c_int32)), ("source", C.POINTER(C.c_uint8)), ("cap_tokens", C.c_int32), ("n_tokens", C.c_int32),
        ("round_drafted", C.POINTER(C.c_int32)), ("round_accepted", C.POINTER(C.c_int32)),
        ("cap_rounds", C.c_int32), ("n_rounds", C.c_int32),
        ("kv_len_small", C.c_int32), ("kv_len_large", C.c_int32), ("n_drafted", C.c_int32), ("n_accepted", C.c_int32),
        ("draft_tokens", C.POINTER(C.c_int32)), ("draft_argmax", C.POINTER(C.c_int32)), ("cap_drafts", C.c_int32),
        ("choice_argmax", C.POINTER(C.c_int32)),
        ("seconds", C.c_double), ("bytes_algorithmic", C.c_int64),
    ]


EXPORTS = [
    "st_model_create", "st_model_destroy", "st_seq_alloc", "st_seq_free", "st_seq_reserve", "st_kv_len",
    "st_kv_truncate", "st_prefill", "st_decode_step", "st_generate_spec", "st_fill_tensor_bf16",
    "st_weight_bytes", "st_kv_bytes_per_token", "st_last_device_status", "st_strerror",
    "st_kernel_launches", "st_time_gemv", "st_argmax_static", "st_generate_spec_batch", "st_decode_geometry",
    "st_generate_specdec", "st_selftest_bounded_wait",
]

_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with paper_2504_12329_b200/build.py "
                              "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(LIB_PATH)
        L.st_model_create.restype = C.c_int
        L.st_model_create.argtypes = [C.POINTER(StConfig), C.c_uint64, C.c_uint32, C.c_void_p, C.POINTER(C.c_void_p)]
        L.st_model_destroy.restype = None
        L.st_model_destroy.argtypes = [C.c_void_p]
        L.st_seq_alloc.restype = C.c_int
        L.st_seq_alloc.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]
        L.st_seq_free.restype = C.c_int
        L.st_seq_free.argtypes = [C.c_void_p, C.c_int32]
        L.st_seq_reserve.restype = C.c_int
        L.st_seq_reserve.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
        L.st_kv_len.restype = C.c_int
        L.st_kv_len.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int32)]
        L.st_kv_truncate.restype = C.c_int
        L.st_kv_truncate.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
        L.st_prefill.restype = C.c_int
        L.st_prefill.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p]
        L.st_decode_step.restype = C.c_int
        L.st_decode_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        L.st_generate_spec.restype = C.c_int
        L.st_generate_spec.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(StSpecParams), C.c_void_p, C.c_int32,
                                       C.c_void_p, C.c_int32, C.POINTER(StSpecResult)]
        L.st_fill_tensor_bf16.restype = C.c_int
        L.st_fill_tensor_bf16.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p]
        L.st_weight_bytes.restype = C.c_int64
        L.st_weight_bytes.argtypes = [C.c_void_p]
        L.st_kv_bytes_per_token.restype = C.c_int64
        L.st_kv_bytes_per_token.argtypes = [C.c_void_p]
        L.st_last_device_status.restype = C.c_int
        L.st_last_device_status.argtypes = [C.c_void_p]
        L.st_kernel_launches.restype = C.c_int64
        L.st_kernel_launches.argtypes = []
        L.st_time_gemv.restype = C.c_int
        L.st_time_gemv.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(C.c_double)]
        L.st_generate_spec_batch.restype = C.c_int
        L.st_generate_spec_batch.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(StSpecParams), C.c_int32, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.st_argmax_static.restype = C.c_int
        L.st_argmax_static.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        L.st_decode_geometry.restype = C.c_int
        L.st_decode_geometry.argtypes = [C.c_void_p, C.c_int32] + [C.POINTER(C.c_int32)] * 4
        L.st_selftest_bounded_wait.restype = C.c_int
        L.st_selftest_bounded_wait.argtypes = [C.c_void_p, C.c_int32]
        L.st_generate_specdec.restype = C.c_int
        L.st_generate_specdec.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(StSpecDecParams), C.c_void_p, C.c_int32,
                                          C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.POINTER(StSpecDecResult)]
        L.st_strerror.restype = C.c_char_p
        L.st_strerror.argtypes = [C.c_int]
        _lib = L
    return _lib


class StError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib().st_strerror(status).decode()} ({status})")


def _check(rc: int, where: str):
    if rc != ST_OK:
        raise StError(rc, where)


def st_kernel_launches() -> int:
    return lib().st_kernel_launches()


def st_argmax_static(logits, n: int, argmax_out, stream: int = 0):
    """Lowest-id argmax of a device fp32 vector into a device int32, using only the library's built-in
    scratch array (no allocation anywhere on the path)."""
    _check(lib().st_argmax_static(_dev_ptr(logits), n, _dev_ptr(argmax_out), C.c_void_p(stream)), "st_argmax_static")


def st_strerror(status: int) -> str:
    return lib().st_strerror(status).decode()


def _np_ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dev_ptr(t):
    """Device pointer of a torch CUDA tensor (or None)."""
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return C.c_void_p(t.data_ptr())


class _TorchAllocator:
    """Allocator hooks that serve the library's device memory from PyTorch's caching allocator."""

    def __init__(self, device):
        import torch
        self._torch = torch
        self.device = device
        self.live = {}
        self.alloc_cb = ALLOC_FN(self._alloc)
        self.free_cb = FREE_FN(self._free)

    def _alloc(self, nbytes, _user):
        try:
            t = self._torch.empty(int(nbytes), dtype=self._torch.uint8, device=self.device)
        except Exception:
            return None
        self.live[t.data_ptr()] = t
        return t.data_ptr()

    def _free(self, ptr, _user):
        self.live.pop(ptr, None)


def st_fill_tensor_bf16(seed: int, tag: int, tid: int, idx0: int, n: int, out, stream: int = 0):
    """out: torch CUDA tensor of n 16-bit elements (bf16 or int16)."""
    _check(lib().st_fill_tensor_bf16(seed, tag, tid, idx0, n, _dev_ptr(out), C.c_void_p(stream)), "st_fill_tensor_bf16")


@dataclass
class SpecResult:
    tokens: np.ndarray
    source: np.ndarray
    handoffs: list
    emission_tokens: np.ndarray
    emission_source: np.ndarray
    emission_fed: np.ndarray
    emission_argmax: np.ndarray
    kv_len_small: int
    kv_len_large: int
    logits_trace: np.ndarray | None
    seconds: float
    bytes_algorithmic: int
    n_steps: int
    handoff_kinds: list = None   # 1 reflection / affirmation / every-delimiter, 2 verification, 3 excessive reflection
    phase_times: dict = None     # kind of pass -> (device seconds, passes): prompt_prefill, catchup, decode


class Model:
    """One transformer on the current CUDA device (st_model_create / st_model_destroy)."""

    def __init__(self, shape: dict, *, seed: int = 0, tag: int = 0, max_seqs: int = 1, max_tokens: int = 4096,
                 page_size: int = 64, stream: int | None = None, torch_alloc: bool = True):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: the library has no CPU path")
        self._torch = torch
        self.device = torch.device("cuda", torch.cuda.current_device())
        self.stream = torch.cuda.current_stream().cuda_stream if stream is None else stream
        self._allocator = _TorchAllocator(self.device) if torch_alloc else None
        cfg = StConfig()
        for k in ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "vocab", "tie_embeddings", "qkv_bias"):
            setattr(cfg, k, int(shape[k]))
        cfg.rope_theta = float(shape["rope_theta"])
        cfg.rms_eps = float(shape["rms_eps"])
        cfg.max_seqs, cfg.max_tokens, cfg.page_size = max_seqs, max_tokens, page_size
        if self._allocator:
            cfg.alloc, cfg.free = self._allocator.alloc_cb, self._allocator.free_cb
        self.cfg = cfg
        self.vocab = cfg.vocab
        h = C.c_void_p()
        _check(lib().st_model_create(C.byref(cfg), seed, tag, C.c_void_p(self.stream), C.byref(h)), "st_model_create")
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            lib().st_model_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # --- sequences -------------------------------------------------------------------------
    def st_seq_alloc(self) -> int:
        s = C.c_int32()
        _check(lib().st_seq_alloc(self.h, C.byref(s)), "st_seq_alloc")
        return s.value

    def st_seq_free(self, slot: int):
        _check(lib().st_seq_free(self.h, slot), "st_seq_free")

    def st_seq_reserve(self, slot: int, n_tokens: int):
        _check(lib().st_seq_reserve(self.h, slot, n_tokens), "st_seq_reserve")

    def st_kv_len(self, slot: int) -> int:
        n = C.c_int32()
        _check(lib().st_kv_len(self.h, slot, C.byref(n)), "st_kv_len")
        return n.value

    def st_kv_truncate(self, slot: int, new_len: int):
        _check(lib().st_kv_truncate(self.h, slot, new_len), "st_kv_truncate")

    def st_selftest_bounded_wait(self, which: int) -> int:
        """Status code of the bounded-wait self-test (ST_ERR_TIMEOUT is the expected outcome)."""
        return int(lib().st_selftest_bounded_wait(self.h, which))

    def st_decode_geometry(self, ctx: int) -> dict:
        """Attention layout of the single-kernel decode step with ctx tokens cached (host arithmetic)."""
        v = [C.c_int32() for _ in range(4)]
        _check(lib().st_decode_geometry(self.h, ctx, *[C.byref(x) for x in v]), "st_decode_geometry")
        return dict(n_splits=v[0].value, kv_cap=v[1].value, max_chunks=v[2].value, own_chunk_empty=bool(v[3].value))

    # --- passes ----------------------------------------------------------------------------
    def st_prefill(self, slot: int, tokens, last_logits=None):
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        _check(lib().st_prefill(self.h, slot, _np_ptr(t), t.size, _dev_ptr(last_logits)), "st_prefill")

    def st_decode_step(self, slots, tokens_dev, logits=None, argmax=None):
        s = np.ascontiguousarray(slots, dtype=np.int32)
        _check(lib().st_decode_step(self.h, _np_ptr(s), _dev_ptr(tokens_dev), s.size, _dev_ptr(logits), _dev_ptr(argmax)),
               "st_decode_step")

    def st_weight_bytes(self) -> int:
        return lib().st_weight_bytes(self.h)

    def st_kv_bytes_per_token(self) -> int:
        return lib().st_kv_bytes_per_token(self.h)

    def st_time_gemv(self, which: int, iters: int) -> float:
        sec = C.c_double()
        _check(lib().st_time_gemv(self.h, which, iters, C.byref(sec)), "st_time_gemv")
        return sec.value

    def st_last_device_status(self) -> int:
        return lib().st_last_device_status(self.h)


class _ResultBuffers:
    """Host buffers of one st_spec_result and the struct that points at them."""

    def __init__(self, max_new_tokens, vocab_limit, trace_first_step, trace_n_steps, cap_steps, cap_handoffs):
        self.cap_steps = 2 * max_new_tokens + 8 if cap_steps is None else cap_steps
        self.cap_handoffs = max_new_tokens + 1 if cap_handoffs is None else cap_handoffs
        self.tokens = np.zeros(max_new_tokens + 1, dtype=np.int32)
        self.source = np.zeros(max_new_tokens + 1, dtype=np.uint8)
        self.hand = (StHandoff * max(self.cap_handoffs, 1))()
        self.kinds = np.zeros(max(self.cap_handoffs, 1), dtype=np.uint8)
        n = max(self.cap_steps, 1)
        self.e_tok, self.e_fed, self.e_arg = (np.zeros(n, dtype=np.int32) for _ in range(3))
        self.e_src = np.zeros(n, dtype=np.uint8)
        self.trace = np.zeros((trace_n_steps, vocab_limit), dtype=np.float32) if trace_n_steps > 0 else None
        self.trace_first_step, self.trace_n_steps = trace_first_step, trace_n_steps

    def fill(self, R: StSpecResult):
        R.tokens = self.tokens.ctypes.data_as(C.POINTER(C.c_int32))
        R.source = self.source.ctypes.data_as(C.POINTER(C.c_uint8))
        R.cap_tokens = self.tokens.size
        R.handoffs = C.cast(self.hand, C.POINTER(StHandoff))
        R.cap_handoffs = self.cap_handoffs
        R.handoff_kinds = self.kinds.ctypes.data_as(C.POINTER(C.c_uint8))
        R.emission_tokens = self.e_tok.ctypes.data_as(C.POINTER(C.c_int32))
        R.emission_source = self.e_src.ctypes.data_as(C.POINTER(C.c_uint8))
        R.emission_fed = self.e_fed.ctypes.data_as(C.POINTER(C.c_int32))
        R.emission_argmax = self.e_arg.ctypes.data_as(C.POINTER(C.c_int32))
        R.cap_steps = self.cap_steps
        R.logits_trace = self.trace.ctypes.data_as(C.POINTER(C.c_float)) if self.trace is not None else None
        R.trace_first_step = self.trace_first_step
        R.trace_n_steps = self.trace_n_steps

    def result(self, R: StSpecResult) -> SpecResult:
        n, s = R.n_tokens, min(R.n_steps, self.cap_steps)
        return SpecResult(self.tokens[:n].copy(), self.source[:n].copy(),
                          [(self.hand[i].seg_start, self.hand[i].step, self.hand[i].catchup_len)
                           for i in range(min(R.n_handoffs, self.cap_handoffs))],
                          self.e_tok[:s].copy(), self.e_src[:s].copy(), self.e_fed[:s].copy(), self.e_arg[:s].copy(),
                          R.kv_len_small, R.kv_len_large, self.trace, R.seconds, R.bytes_algorithmic, R.n_steps,
                          self.kinds[:min(R.n_handoffs, self.cap_handoffs)].tolist(),
                          {"prompt_prefill": (R.t_prompt_prefill_s, R.n_prompt_prefill), "catchup": (R.t_catchup_s, R.n_catchup),
                           "decode": (R.t_decode_s, R.n_decode)})


def _spec_params(delimiter_id, keyword_ids, n1, keep_probe, eos_id, vocab_limit, max_new_tokens, takeover_every_delimiter,
                 target_first_n, affirmation_ids=(), verification_ids=(), n2=125, neg_threshold=-1, n3=125, aux_ids=(),
                 probe_len=1, delimiter_ids=(), temperature=0.0, sample_seed=0, top_p=0.0):
    """st_spec_params and the arrays it points at (keep both alive during the call)."""
    arrs = [np.ascontiguousarray(a, dtype=np.int32) for a in (keyword_ids, affirmation_ids, verification_ids, aux_ids, delimiter_ids)]
    ip = lambda a: a.ctypes.data_as(C.POINTER(C.c_int32))
    kw, aff, ver, aux, dl = arrs
    P = StSpecParams(delimiter_id, ip(kw), kw.size, n1, int(keep_probe), eos_id, vocab_limit, max_new_tokens,
                     int(takeover_every_delimiter), int(target_first_n), ip(aff), aff.size, ip(ver), ver.size, n2,
                     neg_threshold, n3, ip(aux), aux.size, probe_len, ip(dl), dl.size, float(temperature), int(sample_seed), float(top_p))
    return P, arrs


def st_generate_spec(small: Model, large: Model | None, prompt, *, delimiter_id: int, keyword_ids, n1: int = 20,
                     keep_probe: bool = False, eos_id: int = -1, vocab_limit: int = 0, max_new_tokens: int,
                     force=None, trace_first_step: int = 0, trace_n_steps: int = 0, cap_steps: int | None = None,
                     cap_handoffs: int | None = None, takeover_every_delimiter: bool = False,
                     target_first_n: int = 0, **rules) -> SpecResult:
    """Host buffers in, host buffers out: marshals the arguments of st_generate_spec.  rules: affirmation_ids,
    verification_ids, n2, neg_threshold, n3, aux_ids (the other takeovers of the paper's Section 3)."""
    prompt = np.ascontiguousarray(prompt, dtype=np.int32)
    P, _keep = _spec_params(delimiter_id, keyword_ids, n1, keep_probe, eos_id, vocab_limit, max_new_tokens,
                            takeover_every_delimiter, target_first_n, **rules)
    if vocab_limit <= 0:
        vocab_limit = small.vocab if large is None else min(small.vocab, large.vocab)
    if cap_steps is None:   # replaced probe sentences are steps that leave no token
        cap_steps = (1 + max(1, int(rules.get("probe_len", 1)))) * max_new_tokens + 8
    bufs = _ResultBuffers(max_new_tokens, vocab_limit, trace_first_step, trace_n_steps, cap_steps, cap_handoffs)
    R = StSpecResult()
    bufs.fill(R)
    f = None if force is None else np.ascontiguousarray(force, dtype=np.int32)
    rc = lib().st_generate_spec(small.h, large.h if large is not None else None, C.byref(P), _np_ptr(prompt), prompt.size,
                                _np_ptr(f), 0 if f is None else f.size, C.byref(R))
    _check(rc, "st_generate_spec")
    return bufs.result(R)


def st_generate_spec_batch(small: Model, large: Model | None, prompts, *, delimiter_id: int, keyword_ids, n1: int = 20,
                           keep_probe: bool = False, eos_id: int = -1, vocab_limit: int = 0, max_new_tokens,
                           forces=None, takeover_every_delimiter: bool = False, target_first_n: int = 0, **rules) -> list:
    """prompts / forces: lists of per-sequence arrays; max_new_tokens: one int or a list per sequence."""
    n = len(prompts)
    budgets = [int(max_new_tokens)] * n if np.isscalar(max_new_tokens) else [int(x) for x in max_new_tokens]
    P, _keep = _spec_params(delimiter_id, keyword_ids, n1, keep_probe, eos_id, vocab_limit, max(budgets) if budgets else 0,
                            takeover_every_delimiter, target_first_n, **rules)
    if vocab_limit <= 0:
        vocab_limit = small.vocab if large is None else min(small.vocab, large.vocab)
    flat_p = np.ascontiguousarray(np.concatenate([np.asarray(p, dtype=np.int32) for p in prompts]) if n else np.zeros(0, np.int32))
    off_p = np.zeros(n + 1, dtype=np.int32)
    off_p[1:] = np.cumsum([len(p) for p in prompts])
    flat_f = off_f = None
    if forces is not None:
        flat_f = np.ascontiguousarray(np.concatenate([np.asarray(f, dtype=np.int32) for f in forces]))
        off_f = np.zeros(n + 1, dtype=np.int32)
        off_f[1:] = np.cumsum([len(f) for f in forces])
    budget_arr = np.ascontiguousarray(budgets, dtype=np.int32)
    k = 1 + max(1, int(rules.get("probe_len", 1)))
    bufs = [_ResultBuffers(b, vocab_limit, 0, 0, k * b + 8, None) for b in budgets]
    Rs = (StSpecResult * max(n, 1))()
    for i, b in enumerate(bufs):
        b.fill(Rs[i])
    rc = lib().st_generate_spec_batch(small.h, large.h if large is not None else None, C.byref(P), n, _np_ptr(flat_p),
                                      _np_ptr(off_p), _np_ptr(budget_arr), _np_ptr(flat_f), _np_ptr(off_f),
                                      C.cast(Rs, C.c_void_p))
    _check(rc, "st_generate_spec_batch")
    return [b.result(Rs[i]) for i, b in enumerate(bufs)]


@dataclass
class SpecDecResult:
    tokens: np.ndarray
    source: np.ndarray          # 0 = accepted draft, 1 = written by the target
    rounds: list                # (drafted, accepted) per round
    kv_len_small: int
    kv_len_large: int
    n_drafted: int
    n_accepted: int
    draft_tokens: np.ndarray
    draft_argmax: np.ndarray
    choice_argmax: np.ndarray
    seconds: float
    bytes_algorithmic: int


def st_generate_specdec(small: Model, large: Model, prompt, *, gamma: int = 20, eos_id: int = -1, vocab_limit: int = 0,
                        max_new_tokens: int, force_draft=None, force_target=None) -> SpecDecResult:
    """Greedy speculative decoding (the paper's comparison system): marshals the arguments of st_generate_specdec."""
    prompt = np.ascontiguousarray(prompt, dtype=np.int32)
    P = StSpecDecParams(gamma, eos_id, vocab_limit, max_new_tokens)
    n = max_new_tokens + 1
    ip = lambda a: a.ctypes.data_as(C.POINTER(C.c_int32))
    tokens, source = np.zeros(n, dtype=np.int32), np.zeros(n, dtype=np.uint8)
    rd, ra, ca = np.zeros(n, dtype=np.int32), np.zeros(n, dtype=np.int32), np.zeros(n, dtype=np.int32)
    cap_drafts = gamma * n
    dt, da = np.zeros(cap_drafts, dtype=np.int32), np.zeros(cap_drafts, dtype=np.int32)
    R = StSpecDecResult()
    R.tokens, R.source, R.cap_tokens = ip(tokens), source.ctypes.data_as(C.POINTER(C.c_uint8)), n
    R.round_drafted, R.round_accepted, R.cap_rounds = ip(rd), ip(ra), n
    R.draft_tokens, R.draft_argmax, R.cap_drafts, R.choice_argmax = ip(dt), ip(da), cap_drafts, ip(ca)
    fd = None if force_draft is None else np.ascontiguousarray(force_draft, dtype=np.int32)
    ft = None if force_target is None else np.ascontiguousarray(force_target, dtype=np.int32)
    rc = lib().st_generate_specdec(small.h, large.h, C.byref(P), _np_ptr(prompt), prompt.size, _np_ptr(fd), 0 if fd is None else fd.size,
                                   _np_ptr(ft), 0 if ft is None else ft.size, C.byref(R))
    _check(rc, "st_generate_specdec")
    k = R.n_rounds
    return SpecDecResult(tokens[:R.n_tokens].copy(), source[:R.n_tokens].copy(), list(zip(rd[:k].tolist(), ra[:k].tolist())),
                         R.kv_len_small, R.kv_len_large, R.n_drafted, R.n_accepted, dt[:R.n_drafted].copy(), da[:R.n_drafted].copy(),
                         ca[:R.n_tokens].copy(), R.seconds, R.bytes_algorithmic)
