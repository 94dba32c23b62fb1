"""ctypes binding of the CPU oracle (oracle/st_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
CPU-baseline leg of the benchmark.  Nothing here touches the CUDA library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "st_oracle.c")
_LIB = os.path.join(_HERE, "libst_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, OpenMP over output rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


class Config(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("hidden", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("ffn", C.c_int32), ("vocab", C.c_int32),
        ("rope_theta", C.c_double), ("rms_eps", C.c_double),
        ("tie_embeddings", C.c_int32), ("qkv_bias", C.c_int32),
    ]


class _SpecParams(C.Structure):
    _fields_ = [
        ("delimiter_id", C.c_int32), ("keyword_ids", C.POINTER(C.c_int32)), ("n_keywords", C.c_int32),
        ("n1", C.c_int32), ("keep_probe", C.c_int32), ("eos_id", C.c_int32), ("vocab_limit", C.c_int32),
        ("max_new_tokens", C.c_int32),
        ("takeover_every_delimiter", C.c_int32), ("target_first_n", C.c_int32),
        ("affirmation_ids", C.POINTER(C.c_int32)), ("n_affirmation", C.c_int32),
        ("verification_ids", C.POINTER(C.c_int32)), ("n_verification", C.c_int32),
        ("n2", C.c_int32), ("neg_threshold", C.c_int32), ("n3", C.c_int32),
        ("aux_ids", C.POINTER(C.c_int32)), ("n_aux", C.c_int32), ("probe_len", C.c_int32),
        ("delimiter_ids", C.POINTER(C.c_int32)), ("n_delimiters", C.c_int32),
        ("temperature", C.c_double), ("sample_seed", C.c_uint64), ("top_p", C.c_double),
    ]


class _Handoff(C.Structure):
    _fields_ = [("seg_start", C.c_int32), ("step", C.c_int32), ("catchup_len", C.c_int32)]


class _SpecResult(C.Structure):
    _fields_ = [
        ("tokens", C.POINTER(C.c_int32)), ("source", C.POINTER(C.c_uint8)),
        ("cap_tokens", C.c_int32), ("n_tokens", C.c_int32),
        ("handoffs", C.POINTER(_Handoff)), ("cap_handoffs", C.c_int32), ("n_handoffs", C.c_int32),
        ("emission_tokens", C.POINTER(C.c_int32)), ("emission_source", C.POINTER(C.c_uint8)),
        ("emission_fed", C.POINTER(C.c_int32)), ("emission_argmax", C.POINTER(C.c_int32)),
        ("emission_margin", C.POINTER(C.c_double)),
        ("cap_steps", C.c_int32), ("n_steps", C.c_int32),
        ("kv_len_small", C.c_int32), ("kv_len_large", C.c_int32),
        ("logits_trace", C.POINTER(C.c_double)), ("trace_first_step", C.c_int32), ("trace_n_steps", C.c_int32),
        ("handoff_kinds", C.POINTER(C.c_uint8)),
    ]


class _SpecDecParams(C.Structure):
    _fields_ = [("gamma", C.c_int32), ("eos_id", C.c_int32), ("vocab_limit", C.c_int32), ("max_new_tokens", C.c_int32)]


class _SpecDecResult(C.Structure):
    _fields_ = [
        ("tokens", C.POINTER(C.c_int32)), ("source", C.POINTER(C.c_uint8)), ("cap_tokens", C.c_int32), ("n_tokens", C.c_int32),
        ("round_drafted", C.POINTER(C.c_int32)), ("round_accepted", C.POINTER(C.c_int32)),
        ("cap_rounds", C.c_int32), ("n_rounds", C.c_int32),
        ("kv_len_small", C.c_int32), ("kv_len_large", C.c_int32), ("n_drafted", C.c_int32), ("n_accepted", C.c_int32),
        ("choice_margin", C.POINTER(C.c_double)), ("draft_margin", C.POINTER(C.c_double)), ("cap_drafts", C.c_int32),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_sm64_mix.restype = C.c_uint64
        L.orc_sm64_mix.argtypes = [C.c_uint64]
        L.orc_sm64_nth.restype = C.c_uint64
        L.orc_sm64_nth.argtypes = [C.c_uint64, C.c_uint64]
        L.orc_stream_key.restype = C.c_uint64
        L.orc_stream_key.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32]
        L.orc_round_bf16.restype = C.c_float
        L.orc_round_bf16.argtypes = [C.c_float]
        L.orc_fill_tensor.restype = None
        L.orc_fill_tensor.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64, C.c_uint64, C.c_void_p]
        L.orc_model_create.restype = C.c_void_p
        L.orc_model_create.argtypes = [C.POINTER(Config), C.c_uint64, C.c_uint32, C.c_int]
        L.orc_model_destroy.restype = None
        L.orc_model_destroy.argtypes = [C.c_void_p]
        L.orc_model_set_tensor.restype = C.c_int
        L.orc_model_set_tensor.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_uint64]
        L.orc_model_set_gain.restype = C.c_int
        L.orc_model_set_gain.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p]
        L.orc_rmsnorm.restype = None
        L.orc_rmsnorm.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_double, C.c_void_p]
        L.orc_rope.restype = None
        L.orc_rope.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_double]
        L.orc_silu.restype = C.c_double
        L.orc_silu.argtypes = [C.c_double]
        L.orc_attend.restype = None
        L.orc_attend.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_int64, C.c_void_p]
        L.orc_kv_create.restype = C.c_void_p
        L.orc_kv_create.argtypes = [C.c_void_p, C.c_int64]
        L.orc_kv_destroy.restype = None
        L.orc_kv_destroy.argtypes = [C.c_void_p]
        L.orc_kv_len.restype = C.c_int64
        L.orc_kv_len.argtypes = [C.c_void_p]
        L.orc_kv_truncate.restype = None
        L.orc_kv_truncate.argtypes = [C.c_void_p, C.c_int64]
        L.orc_forward.restype = C.c_int
        L.orc_forward.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p]
        L.orc_forward_last.restype = C.c_int
        L.orc_forward_last.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
        L.orc_forward_full.restype = C.c_int
        L.orc_forward_full.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
        L.orc_argmax.restype = C.c_int32
        L.orc_argmax.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_double)]
        L.orc_sample.restype = C.c_int32
        L.orc_sample.argtypes = [C.c_void_p, C.c_int32, C.c_double, C.c_uint64, C.c_uint32, C.POINTER(C.c_double)]
        L.orc_nucleus_threshold.restype = C.c_double
        L.orc_nucleus_threshold.argtypes = [C.c_void_p, C.c_int32, C.c_double, C.c_double, C.POINTER(C.c_double)]
        L.orc_sample_top_p.restype = C.c_int32
        L.orc_sample_top_p.argtypes = [C.c_void_p, C.c_int32, C.c_double, C.c_double, C.c_uint64, C.c_uint32,
                                       C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.orc_gumbel.restype = C.c_double
        L.orc_gumbel.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32]
        L.orc_generate_specdec.restype = C.c_int
        L.orc_generate_specdec.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(_SpecDecParams), C.c_void_p, C.c_int32,
                                           C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.POINTER(_SpecDecResult)]
        L.orc_generate_spec.restype = C.c_int
        L.orc_generate_spec.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(_SpecParams), C.c_void_p, C.c_int32,
                                        C.c_void_p, C.c_int32, C.POINTER(_SpecResult)]
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


# Tensor selectors for Model.set_tensor (layer-local ids of the C file).
WQ, WK, WV, BQ, BK, BV, WO, WG, WU, WD = 1, 2, 3, 4, 5, 6, 7, 9, 10, 11
EMBED, LMHEAD = 0, 1


def fill_tensor(seed: int, tag: int, tid: int, idx0: int, n: int) -> np.ndarray:
    """Seeded weights: elements idx0..idx0+n-1 of tensor `tid` of model `tag` (bf16 values as float32)."""
    out = np.empty(n, dtype=np.float32)
    lib().orc_fill_tensor(seed, tag, tid, idx0, n, _p(out))
    return out


def layer_tid(layer: int, which: int) -> int:
    return 16 * (layer + 1) + which


def rmsnorm(x, g=None, eps=1e-6):
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.empty_like(x)
    gp = None if g is None else _p(np.ascontiguousarray(g, dtype=np.float64))
    lib().orc_rmsnorm(_p(x), gp, x.size, eps, _p(y))
    return y


def rope(x, pos: int, theta: float):
    y = np.array(x, dtype=np.float64, copy=True)
    lib().orc_rope(_p(y), y.size, pos, theta)
    return y


def silu(z: float) -> float:
    return lib().orc_silu(z)


def attend(q, k, v):
    """softmax(q k^T / sqrt(d)) v for one query; k, v: [n, d]."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    k = np.ascontiguousarray(k, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    out = np.empty(q.size, dtype=np.float64)
    lib().orc_attend(_p(q), _p(k), _p(v), k.shape[0], q.size, k.shape[1], _p(out))
    return out


def argmax(z, limit=None):
    z = np.ascontiguousarray(z, dtype=np.float64)
    m = C.c_double()
    i = lib().orc_argmax(_p(z), z.size if limit is None else limit, C.byref(m))
    return int(i), float(m.value)


def sample(z, temperature: float, seed: int, step: int, limit=None):
    """(token, margin of the perturbed values) of the Gumbel-max sampler."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    m = C.c_double()
    i = lib().orc_sample(_p(z), z.size if limit is None else limit, temperature, seed, step, C.byref(m))
    return int(i), float(m.value)


def nucleus_threshold(z, temperature: float, top_p: float, limit=None):
    """(threshold logit, gap): the nucleus of softmax(z / T) is {i: z[i] >= threshold}."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    g = C.c_double()
    t = lib().orc_nucleus_threshold(_p(z), z.size if limit is None else limit, temperature, top_p, C.byref(g))
    return float(t), float(g.value)


def sample_top_p(z, temperature: float, top_p: float, seed: int, step: int, limit=None):
    """(token, margin of the perturbed values, gap of the nucleus cut) of the Gumbel-max sampler restricted to the nucleus."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    m, g = C.c_double(), C.c_double()
    i = lib().orc_sample_top_p(_p(z), z.size if limit is None else limit, temperature, top_p, seed, step, C.byref(m), C.byref(g))
    return int(i), float(m.value), float(g.value)


def gumbel(seed: int, step: int, i: int) -> float:
    return float(lib().orc_gumbel(seed, step, i))


class Model:
    def __init__(self, cfg: Config, seed: int, tag: int, materialize: bool = True):
        self.cfg = cfg
        self.h = lib().orc_model_create(C.byref(cfg), seed, tag, int(materialize))
        if not self.h:
            raise RuntimeError("orc_model_create failed")

    def close(self):
        if self.h:
            lib().orc_model_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except TypeError:   # interpreter shutdown: module globals are already gone
            pass

    def set_tensor(self, layer: int, which: int, data):
        a = np.ascontiguousarray(data, dtype=np.float32)
        if lib().orc_model_set_tensor(self.h, layer, which, _p(a), a.size) != 0:
            raise ValueError("tensor size mismatch")

    def set_gain(self, layer: int, which: int, g):
        a = np.ascontiguousarray(g, dtype=np.float64)
        assert a.size == self.cfg.hidden
        lib().orc_model_set_gain(self.h, layer, which, _p(a))

    def forward_full(self, tokens) -> np.ndarray:
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        out = np.empty((t.size, self.cfg.vocab), dtype=np.float64)
        lib().orc_forward_full(self.h, _p(t), t.size, _p(out))
        return out


class KV:
    def __init__(self, model: Model, cap: int):
        self.model = model
        self.h = lib().orc_kv_create(model.h, cap)
        if not self.h:
            raise MemoryError("orc_kv_create failed")

    def close(self):
        if self.h:
            lib().orc_kv_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except TypeError:   # interpreter shutdown: module globals are already gone
            pass

    def __len__(self):
        return int(lib().orc_kv_len(self.h))

    def truncate(self, n: int):
        lib().orc_kv_truncate(self.h, n)

    def forward(self, tokens, all_rows: bool = False) -> np.ndarray:
        """Feed tokens at the next positions; logits of the last row ([vocab]) or of all rows."""
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        V = self.model.cfg.vocab
        out = np.empty((t.size, V) if all_rows else (V,), dtype=np.float64)
        rc = lib().orc_forward(self.model.h, self.h, _p(t), t.size, int(all_rows), _p(out))
        if rc != 0:
            raise RuntimeError(f"orc_forward rc={rc}")
        return out

    def forward_last(self, tokens) -> np.ndarray:
        """forward(tokens) with the last layer's attention and FFN evaluated only for the last row (the only row
        the returned logits depend on); keys and values of every row are cached as usual."""
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        out = np.empty((self.model.cfg.vocab,), dtype=np.float64)
        rc = lib().orc_forward_last(self.model.h, self.h, _p(t), t.size, _p(out))
        if rc != 0:
            raise RuntimeError(f"orc_forward_last rc={rc}")
        return out


@dataclass
class SpecResult:
    tokens: np.ndarray
    source: np.ndarray
    handoffs: list            # (seg_start, step, catchup_len)
    emission_tokens: np.ndarray
    emission_source: np.ndarray
    emission_fed: np.ndarray
    emission_argmax: np.ndarray
    emission_margin: np.ndarray
    kv_len_small: int
    kv_len_large: int
    logits_trace: np.ndarray | None
    rc: int
    handoff_kinds: list = None   # 1 reflection / affirmation, 2 verification, 3 excessive reflection


def generate_spec(small: Model, large: Model | None, prompt, *, delimiter_id: int, keyword_ids, n1: int = 20,
                  keep_probe: bool = False, eos_id: int = -1, vocab_limit: int = 0, max_new_tokens: int,
                  force=None, trace_first_step: int = 0, trace_n_steps: int = 0,
                  takeover_every_delimiter: bool = False, target_first_n: int = 0, affirmation_ids=(),
                  verification_ids=(), n2: int = 125, neg_threshold: int = -1, n3: int = 125, aux_ids=(),
                  probe_len: int = 1, delimiter_ids=(), temperature: float = 0.0, sample_seed: int = 0,
                  top_p: float = 0.0) -> SpecResult:
    prompt = np.ascontiguousarray(prompt, dtype=np.int32)
    aff = np.ascontiguousarray(affirmation_ids, dtype=np.int32)
    ver = np.ascontiguousarray(verification_ids, dtype=np.int32)
    aux = np.ascontiguousarray(aux_ids, dtype=np.int32)
    dl = np.ascontiguousarray(delimiter_ids, dtype=np.int32)
    ip = lambda a: a.ctypes.data_as(C.POINTER(C.c_int32))
    kw = np.ascontiguousarray(keyword_ids, dtype=np.int32)
    if vocab_limit <= 0:
        vocab_limit = small.cfg.vocab if large is None else min(small.cfg.vocab, large.cfg.vocab)
    P = _SpecParams(delimiter_id, kw.ctypes.data_as(C.POINTER(C.c_int32)), kw.size, n1, int(keep_probe), eos_id,
                    vocab_limit, max_new_tokens, int(takeover_every_delimiter), int(target_first_n),
                    ip(aff), aff.size, ip(ver), ver.size, n2, neg_threshold, n3, ip(aux), aux.size, probe_len,
                    ip(dl), dl.size, float(temperature), int(sample_seed), float(top_p))
    cap_steps = (1 + max(1, probe_len)) * max_new_tokens + 8   # replaced probe sentences are steps without tokens
    tokens = np.zeros(max_new_tokens + 1, dtype=np.int32)
    source = np.zeros(max_new_tokens + 1, dtype=np.uint8)
    hand = (_Handoff * (max_new_tokens + 1))()
    e_tok = np.zeros(cap_steps, dtype=np.int32)
    e_src = np.zeros(cap_steps, dtype=np.uint8)
    e_fed = np.zeros(cap_steps, dtype=np.int32)
    e_arg = np.zeros(cap_steps, dtype=np.int32)
    e_mar = np.zeros(cap_steps, dtype=np.float64)
    trace = np.zeros((trace_n_steps, vocab_limit), dtype=np.float64) if trace_n_steps > 0 else None
    R = _SpecResult()
    R.tokens = tokens.ctypes.data_as(C.POINTER(C.c_int32))
    R.source = source.ctypes.data_as(C.POINTER(C.c_uint8))
    R.cap_tokens = tokens.size
    R.handoffs = C.cast(hand, C.POINTER(_Handoff))
    R.cap_handoffs = max_new_tokens + 1
    R.emission_tokens = e_tok.ctypes.data_as(C.POINTER(C.c_int32))
    R.emission_source = e_src.ctypes.data_as(C.POINTER(C.c_uint8))
    R.emission_fed = e_fed.ctypes.data_as(C.POINTER(C.c_int32))
    R.emission_argmax = e_arg.ctypes.data_as(C.POINTER(C.c_int32))
    R.emission_margin = e_mar.ctypes.data_as(C.POINTER(C.c_double))
    R.cap_steps = cap_steps
    R.logits_trace = trace.ctypes.data_as(C.POINTER(C.c_double)) if trace is not None else None
    R.trace_first_step = trace_first_step
    R.trace_n_steps = trace_n_steps
    kinds = np.zeros(max_new_tokens + 1, dtype=np.uint8)
    R.handoff_kinds = kinds.ctypes.data_as(C.POINTER(C.c_uint8))
    f = None if force is None else np.ascontiguousarray(force, dtype=np.int32)
    rc = lib().orc_generate_spec(small.h, large.h if large is not None else None, C.byref(P), _p(prompt), prompt.size,
                                 None if f is None else _p(f), 0 if f is None else f.size, C.byref(R))
    n, s = R.n_tokens, R.n_steps
    return SpecResult(tokens[:n].copy(), source[:n].copy(),
                      [(hand[i].seg_start, hand[i].step, hand[i].catchup_len) for i in range(R.n_handoffs)],
                      e_tok[:s].copy(), e_src[:s].copy(), e_fed[:s].copy(), e_arg[:s].copy(), e_mar[:s].copy(),
                      R.kv_len_small, R.kv_len_large, trace, rc, kinds[:R.n_handoffs].tolist())


@dataclass
class SpecDecResult:
    tokens: np.ndarray
    source: np.ndarray          # 0 = accepted draft, 1 = written by the target
    rounds: list                # (drafted, accepted) per round
    kv_len_small: int
    kv_len_large: int
    n_drafted: int
    n_accepted: int
    choice_margin: np.ndarray   # per generated position
    draft_margin: np.ndarray    # per draft
    rc: int


def generate_specdec(small: Model, large: Model, prompt, *, gamma: int = 20, eos_id: int = -1, vocab_limit: int = 0,
                     max_new_tokens: int, force_draft=None, force_target=None) -> SpecDecResult:
    """Greedy speculative decoding (the paper's comparison system): see orc_generate_specdec."""
    prompt = np.ascontiguousarray(prompt, dtype=np.int32)
    if vocab_limit <= 0:
        vocab_limit = min(small.cfg.vocab, large.cfg.vocab)
    P = _SpecDecParams(gamma, eos_id, vocab_limit, max_new_tokens)
    n = max_new_tokens + 1
    tokens, source = np.zeros(n, dtype=np.int32), np.zeros(n, dtype=np.uint8)
    rd, ra = np.zeros(n, dtype=np.int32), np.zeros(n, dtype=np.int32)
    cap_drafts = gamma * n
    cm, dm = np.zeros(n, dtype=np.float64), np.zeros(cap_drafts, dtype=np.float64)
    R = _SpecDecResult()
    ip = lambda a: a.ctypes.data_as(C.POINTER(C.c_int32))
    R.tokens, R.source, R.cap_tokens = ip(tokens), source.ctypes.data_as(C.POINTER(C.c_uint8)), n
    R.round_drafted, R.round_accepted, R.cap_rounds = ip(rd), ip(ra), n
    R.choice_margin, R.draft_margin, R.cap_drafts = cm.ctypes.data_as(C.POINTER(C.c_double)), dm.ctypes.data_as(C.POINTER(C.c_double)), cap_drafts
    fd = None if force_draft is None else np.ascontiguousarray(force_draft, dtype=np.int32)
    ft = None if force_target is None else np.ascontiguousarray(force_target, dtype=np.int32)
    rc = lib().orc_generate_specdec(small.h, large.h, C.byref(P), _p(prompt), prompt.size,
                                    None if fd is None else _p(fd), 0 if fd is None else fd.size,
                                    None if ft is None else _p(ft), 0 if ft is None else ft.size, C.byref(R))
    k = R.n_rounds
    return SpecDecResult(tokens[:R.n_tokens].copy(), source[:R.n_tokens].copy(), list(zip(rd[:k].tolist(), ra[:k].tolist())),
                         R.kv_len_small, R.kv_len_large, R.n_drafted, R.n_accepted, cm[:R.n_tokens].copy(),
                         dm[:R.n_drafted].copy(), rc)
