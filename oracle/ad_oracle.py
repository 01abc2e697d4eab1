"""ctypes front end of the CPU checker in ``ad_oracle.c``.

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's
CPU-baseline leg.  The CUDA library never imports it and it never imports the CUDA library.

The C file is compiled on first use with gcc (``-O3 -ffp-contract=off -fopenmp``) into
``oracle/_build``.  ``real="f32"`` is the checker proper; ``real="f64"`` is the same code built with
double precision, used only to bound the checker's own rounding error.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_BUILD = os.path.join(_HERE, "_build")
_LOCK = threading.Lock()
_LIBS = {}


class _Cfg(C.Structure):
    _fields_ = [(n, C.c_int) for n in
                ("d_model", "n_heads", "d_ffn", "vocab", "n_enc", "n_dec", "max_pos",
                 "bos", "pad", "eos", "mask")] + [("ln_eps", C.c_double)]


class _Trace(C.Structure):
    _fields_ = [("it_k", C.POINTER(C.c_int)), ("it_n", C.POINTER(C.c_int)),
                ("iterations", C.c_int), ("offered", C.c_long)]


def build(real: str = "f32") -> str:
    """Compile the checker if its shared object is missing or older than the source."""
    src = os.path.join(_HERE, "ad_oracle.c")
    out = os.path.join(_BUILD, f"libad_oracle_{real}.so")
    with _LOCK:
        if not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(src):
            os.makedirs(_BUILD, exist_ok=True)
            tmp = out + f".{os.getpid()}.tmp"
            cmd = ["gcc", "-O3", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                   "-DORC_REAL=" + ("double" if real == "f64" else "float"), src, "-o", tmp, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, out)
    return out


def _lib(real: str):
    if real not in _LIBS:
        lib = C.CDLL(build(real))
        vp, ip, rp = C.c_void_p, C.POINTER(C.c_int), C.c_void_p
        sig = {
            "orc_weight_count": (C.c_size_t, [C.POINTER(_Cfg)]),
            "orc_model_create": (vp, [C.POINTER(_Cfg), rp]),
            "orc_model_destroy": (None, [vp]),
            "orc_model_pe": (vp, [vp]),
            "orc_state_create": (vp, [vp, ip, C.c_int, C.c_int]),
            "orc_state_destroy": (None, [vp]),
            "orc_state_len": (C.c_int, [vp]),
            "orc_state_memory": (vp, [vp]),
            "orc_state_reset": (None, [vp]),
            "orc_encode_memory": (None, [vp, ip, C.c_int, rp]),
            "orc_decode_block": (C.c_int, [vp, ip, C.c_int, rp]),
            "orc_decode_full": (None, [vp, rp, C.c_int, ip, C.c_int, C.c_int, rp]),
            "orc_top2": (None, [rp, C.c_int, ip, rp, ip, rp]),
            "orc_accept": (C.c_int, [ip, ip, C.c_int, C.c_int, ip]),
            "orc_suffix_match": (C.c_int, [ip, C.c_int, ip, C.c_int]),
            "orc_verify_block": (C.c_int, [vp, C.c_int, ip, C.c_int, ip, rp, rp, ip]),
            "orc_relaxed_choice": (C.c_int, [rp, C.c_int, C.c_int, C.c_int, C.c_double, ip, rp, rp]),
            "orc_verify_block_pp": (C.c_int, [vp, C.c_int, ip, C.c_int, C.c_int, C.c_double, ip, ip, rp, rp, rp, ip]),
            "orc_gad_pp": (C.c_int, [vp, vp, rp, ip, C.c_int, C.c_int, C.c_int, C.c_double, ip, C.POINTER(_Trace)]),
            "orc_commit": (None, [vp, C.c_int]),
            "orc_greedy": (C.c_int, [vp, C.c_int, ip, rp]),
            "orc_draft_verify_stream": (C.c_int, [vp, ip, C.c_int, C.c_int, ip, C.POINTER(_Trace)]),
            "orc_iad": (C.c_int, [vp, ip, C.c_int, C.c_int, C.c_int, ip, C.POINTER(_Trace)]),
            "orc_nar_draft": (None, [vp, rp, C.c_int, ip, C.c_int, C.c_int, ip, rp]),
            "orc_gad": (C.c_int, [vp, vp, rp, ip, C.c_int, C.c_int, ip, C.POINTER(_Trace)]),
            "orc_linear": (None, [rp, rp, rp, rp, C.c_int, C.c_int, C.c_int]),
            "orc_layernorm": (None, [rp, rp, rp, rp, C.c_int, C.c_int, C.c_double]),
            "orc_attention": (None, [rp, rp, rp, ip, rp, C.c_int, C.c_int, C.c_int, C.c_int]),
            "orc_real_size": (C.c_int, []),
        }
        for name, (res, args) in sig.items():
            f = getattr(lib, name)
            f.restype, f.argtypes = res, args
        _LIBS[real] = lib
    return _LIBS[real]


def _ip(a):
    return a.ctypes.data_as(C.POINTER(C.c_int))


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def set_threads(n: int) -> None:
    """Limit the OpenMP team used by the checker (both precisions)."""
    os.environ["OMP_NUM_THREADS"] = str(n)
    try:
        omp = C.CDLL("libgomp.so.1")
        omp.omp_set_num_threads(int(n))
    except OSError:
        pass


def threads() -> int:
    try:
        omp = C.CDLL("libgomp.so.1")
        return int(omp.omp_get_max_threads())
    except OSError:
        return 1


class Ops:
    """The elementary maps, exposed for the pins."""

    def __init__(self, real="f32"):
        self.lib = _lib(real)
        self.dt = np.float64 if real == "f64" else np.float32

    def _a(self, x):
        return np.ascontiguousarray(x, dtype=self.dt)

    def linear(self, x, W, b=None):
        x, W = self._a(x), self._a(W)
        M, i = x.shape
        o = W.shape[1]
        y = np.empty((M, o), self.dt)
        bb = self._a(b) if b is not None else None
        self.lib.orc_linear(x.ctypes.data, W.ctypes.data, bb.ctypes.data if bb is not None else None,
                            y.ctypes.data, M, i, o)
        return y

    def layernorm(self, x, g, b, eps=1e-5):
        x, g, b = self._a(x), self._a(g), self._a(b)
        y = np.empty_like(x)
        self.lib.orc_layernorm(x.ctypes.data, g.ctypes.data, b.ctypes.data, y.ctypes.data,
                               x.shape[0], x.shape[1], eps)
        return y

    def attention(self, q, k, v, limit, H):
        q, k, v = self._a(q), self._a(k), self._a(v)
        lim = _i32(limit)
        out = np.empty_like(q)
        self.lib.orc_attention(q.ctypes.data, k.ctypes.data, v.ctypes.data, _ip(lim), out.ctypes.data,
                               q.shape[0], k.shape[0], q.shape[1], H)
        return out

    def top2(self, logits):
        lg = self._a(logits)
        i1, i2 = C.c_int(), C.c_int()
        v = np.zeros(2, self.dt)
        self.lib.orc_top2(lg.ctypes.data, lg.shape[0], C.byref(i1), v[0:].ctypes.data, C.byref(i2),
                          v[1:].ctypes.data)
        return i1.value, float(v[0]), i2.value, float(v[1])

    def relaxed_choice(self, logits, draft, beta, tau):
        """Section 3.2.3 on one position's scores: (verified token, met, top-1 margin, decision margin)."""
        lg = self._a(logits).ravel()
        met = C.c_int()
        tm, dm = np.zeros(1, self.dt), np.zeros(1, self.dt)
        tok = self.lib.orc_relaxed_choice(lg.ctypes.data, lg.shape[0], int(draft), int(beta), float(tau),
                                          C.byref(met), tm.ctypes.data, dm.ctypes.data)
        return tok, bool(met.value), float(tm[0]), float(dm[0])

    def accept(self, pred, draft, eos=2):
        p, d = _i32(pred), _i32(draft)
        fin = C.c_int()
        n = self.lib.orc_accept(_ip(p), _ip(d), len(p), eos, C.byref(fin))
        return n, bool(fin.value)

    def suffix_match(self, o, x_with_bos):
        """o = [BOS, o_1..o_j]; x_with_bos = [BOS, x_1..x_n].  Returns i or -1."""
        o, x = _i32(o), _i32(x_with_bos)
        return self.lib.orc_suffix_match(_ip(o), len(o) - 1, _ip(x), len(x) - 1)


def _pack(shape, w, dt):
    """Flat buffer in the order ad_oracle.c documents (every W is [in, out])."""
    parts = [w["emb"]]

    def attn(p):
        for n in ("q", "k", "v", "o"):
            parts.extend([w[f"{p}.{n}.W"], w[f"{p}.{n}.b"]])

    def ln(p):
        parts.extend([w[p + ".g"], w[p + ".b"]])

    def ffn(p):
        parts.extend([w[p + ".ffn1.W"], w[p + ".ffn1.b"], w[p + ".ffn2.W"], w[p + ".ffn2.b"]])

    for l in range(shape.n_enc):
        attn(f"enc.{l}.self"); ln(f"enc.{l}.ln1"); ffn(f"enc.{l}"); ln(f"enc.{l}.ln2")
    for l in range(shape.n_dec):
        attn(f"dec.{l}.self"); ln(f"dec.{l}.ln1"); attn(f"dec.{l}.cross"); ln(f"dec.{l}.ln2")
        ffn(f"dec.{l}"); ln(f"dec.{l}.ln3")
    return np.concatenate([np.asarray(p, dtype=dt).ravel() for p in parts])


class Model:
    """One encoder-decoder Transformer held by the checker."""

    def __init__(self, shape, weights, max_pos=512, real="f32", bos=0, pad=1, eos=2, mask=3, ln_eps=1e-5):
        self.lib = _lib(real)
        self.real = real
        self.dt = np.float64 if real == "f64" else np.float32
        self.shape = shape
        self.cfg = _Cfg(shape.d_model, shape.n_heads, shape.d_ffn, shape.vocab, shape.n_enc, shape.n_dec,
                        max_pos, bos, pad, eos, mask, ln_eps)
        self.flat = _pack(shape, weights, self.dt)
        assert self.flat.size == self.lib.orc_weight_count(C.byref(self.cfg))
        self.h = self.lib.orc_model_create(C.byref(self.cfg), self.flat.ctypes.data)
        self.V, self.d = shape.vocab, shape.d_model
        self.eos, self.bos, self.pad, self.mask = eos, bos, pad, mask
        self.max_pos = max_pos

    def __del__(self):
        if getattr(self, "h", None):
            self.lib.orc_model_destroy(self.h)
            self.h = None

    def pe(self):
        p = C.cast(self.lib.orc_model_pe(self.h), C.POINTER(C.c_double if self.real == "f64" else C.c_float))
        return np.ctypeslib.as_array(p, shape=(self.max_pos, self.d)).copy()

    def encode_memory(self, src):
        src = _i32(src)
        mem = np.empty((len(src), self.d), self.dt)
        self.lib.orc_encode_memory(self.h, _ip(src), len(src), mem.ctypes.data)
        return mem

    def decode_full(self, mem, tokens, causal=True):
        tok = _i32(tokens)
        mem = np.ascontiguousarray(mem, dtype=self.dt)
        lg = np.empty((len(tok), self.V), self.dt)
        self.lib.orc_decode_full(self.h, mem.ctypes.data, mem.shape[0], _ip(tok), len(tok), int(causal),
                                 lg.ctypes.data)
        return lg

    def nar_draft(self, mem, prefix_with_bos, k):
        pre = _i32(prefix_with_bos)
        mem = np.ascontiguousarray(mem, dtype=self.dt)
        draft = np.empty(k, np.int32)
        margin = np.empty(k, self.dt)
        self.lib.orc_nar_draft(self.h, mem.ctypes.data, mem.shape[0], _ip(pre), len(pre) - 1, k, _ip(draft),
                               margin.ctypes.data)
        return draft, margin

    def state(self, src, cap=None):
        return State(self, src, cap if cap is not None else self.max_pos)


class State:
    """Decoding state of one sentence: cross K/V of its source and the self-attention cache."""

    def __init__(self, model, src, cap):
        self.m = model
        self.lib = model.lib
        self.src = _i32(src)
        self.h = self.lib.orc_state_create(model.h, _ip(self.src), len(self.src), cap)
        self.cap = cap

    def __del__(self):
        if getattr(self, "h", None):
            self.lib.orc_state_destroy(self.h)
            self.h = None

    @property
    def len(self):
        return self.lib.orc_state_len(self.h)

    def reset(self):
        self.lib.orc_state_reset(self.h)

    def memory(self):
        p = C.cast(self.lib.orc_state_memory(self.h), C.POINTER(C.c_double if self.m.real == "f64" else C.c_float))
        return np.ctypeslib.as_array(p, shape=(len(self.src), self.m.d)).copy()

    def decode_block(self, tokens):
        tok = _i32(tokens)
        lg = np.empty((len(tok), self.m.V), self.m.dt)
        rc = self.lib.orc_decode_block(self.h, _ip(tok), len(tok), lg.ctypes.data)
        if rc != 0:
            raise ValueError("block does not fit the cache")
        return lg

    def verify_block(self, last, draft, want_logits=False):
        """Returns dict(pred, margin, n, finished[, logits]); does not commit."""
        d = _i32(draft)
        k = len(d)
        pred = np.empty(k, np.int32)
        margin = np.empty(k, self.m.dt)
        lg = np.empty((k, self.m.V), self.m.dt) if want_logits else None
        fin = C.c_int()
        n = self.lib.orc_verify_block(self.h, int(last), _ip(d), k, _ip(pred), margin.ctypes.data,
                                      lg.ctypes.data if lg is not None else None, C.byref(fin))
        if n < 1:
            raise ValueError("verify failed (block does not fit)")
        r = dict(pred=pred, margin=margin, n=n, finished=bool(fin.value))
        if want_logits:
            r["logits"] = lg
        return r

    def verify_block_pp(self, last, draft, beta, tau, want_logits=False):
        """Verification with the relaxed top-beta / tau requirement of Section 3.2.3.
        Returns dict(pred, met, margin, dmargin, n, finished[, logits]); does not commit."""
        d = _i32(draft)
        k = len(d)
        pred, met = np.empty(k, np.int32), np.empty(k, np.int32)
        margin, dmargin = np.empty(k, self.m.dt), np.empty(k, self.m.dt)
        lg = np.empty((k, self.m.V), self.m.dt) if want_logits else None
        fin = C.c_int()
        n = self.lib.orc_verify_block_pp(self.h, int(last), _ip(d), k, int(beta), float(tau), _ip(pred), _ip(met),
                                         margin.ctypes.data, dmargin.ctypes.data,
                                         lg.ctypes.data if lg is not None else None, C.byref(fin))
        if n < 1:
            raise ValueError("verify failed (block does not fit)")
        r = dict(pred=pred, met=met.astype(bool), margin=margin, dmargin=dmargin, n=n, finished=bool(fin.value))
        if want_logits:
            r["logits"] = lg
        return r

    def commit(self, n):
        self.lib.orc_commit(self.h, int(n))

    def _trace(self, max_len):
        itk, itn = np.zeros(max_len + 1, np.int32), np.zeros(max_len + 1, np.int32)
        tr = _Trace(_ip(itk), _ip(itn), 0, 0)
        return tr, itk, itn

    @staticmethod
    def _trace_out(tr, itk, itn):
        return dict(iterations=tr.iterations, offered=int(tr.offered),
                    k=itk[:tr.iterations].copy(), n=itn[:tr.iterations].copy())

    def greedy(self, max_len):
        out = np.empty(max_len, np.int32)
        margin = np.empty(max_len, self.m.dt)
        n = self.lib.orc_greedy(self.h, max_len, _ip(out), margin.ctypes.data)
        return out[:n].copy(), margin[:n].copy()

    def draft_verify_stream(self, stream, kmax, max_len):
        st = _i32(np.concatenate([np.asarray(stream, np.int32), np.full(kmax + 1, self.m.pad, np.int32)]))
        out = np.empty(max_len, np.int32)
        tr, itk, itn = self._trace(max_len)
        n = self.lib.orc_draft_verify_stream(self.h, _ip(st), kmax, max_len, _ip(out), C.byref(tr))
        return out[:n].copy(), self._trace_out(tr, itk, itn)

    def iad(self, kmax, max_len):
        out = np.empty(max_len, np.int32)
        tr, itk, itn = self._trace(max_len)
        n = self.lib.orc_iad(self.h, _ip(self.src), len(self.src), kmax, max_len, _ip(out), C.byref(tr))
        return out[:n].copy(), self._trace_out(tr, itk, itn)

    def gad(self, nar_model, kmax, max_len, override=None):
        out = np.empty(max_len, np.int32)
        tr, itk, itn = self._trace(max_len)
        mem = nar_model.encode_memory(self.src) if nar_model is not None else None
        ov = None
        if override is not None:
            ov = _i32(np.concatenate([np.asarray(override, np.int32), np.full(kmax + 1, self.m.pad, np.int32)]))
        n = self.lib.orc_gad(self.h, nar_model.h if nar_model is not None else None,
                             mem.ctypes.data if mem is not None else None,
                             _ip(ov) if ov is not None else None, kmax, max_len, _ip(out), C.byref(tr))
        return out[:n].copy(), self._trace_out(tr, itk, itn)

    def gad_pp(self, nar_model, kmax, max_len, beta, tau, override=None):
        """Generalized mode with the relaxed verification of Section 3.2.3."""
        out = np.empty(max_len, np.int32)
        tr, itk, itn = self._trace(max_len)
        mem = nar_model.encode_memory(self.src) if nar_model is not None else None
        ov = None
        if override is not None:
            ov = _i32(np.concatenate([np.asarray(override, np.int32), np.full(kmax + 1, self.m.pad, np.int32)]))
        n = self.lib.orc_gad_pp(self.h, nar_model.h if nar_model is not None else None,
                                mem.ctypes.data if mem is not None else None,
                                _ip(ov) if ov is not None else None, kmax, max_len, int(beta), float(tau),
                                _ip(out), C.byref(tr))
        return out[:n].copy(), self._trace_out(tr, itk, itn)
