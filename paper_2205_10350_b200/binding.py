"""Thin ctypes binding of the C ABI in include/aggressive_decoding.h.

Argument marshalling only: every step of the decoding path runs inside the CUDA library.  PyTorch
provides device memory (weights, workspace) and the stream.  There is no CPU fallback: if the shared
library is missing, importing this module's loader raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("AD_LIB_PATH", os.path.join(_HERE, "libad_b200.so"))

AD_OK, AD_ERR_ARG, AD_ERR_STATE, AD_ERR_CAPACITY, AD_ERR_TIMEOUT, AD_ERR_CUDA = 0, -1, -2, -3, -4, -5
AD_DTYPE_FP32, AD_DTYPE_BF16 = 0, 1
AD_MODE_IAD, AD_MODE_GAD = 0, 1

EXPORTS = [
    "ad_weight_counts", "ad_query_workspace", "ad_create", "ad_destroy", "ad_last_error", "ad_encode",
    "ad_verify_block", "ad_commit", "ad_force_commit", "ad_generate", "ad_draft_block", "ad_get_state", "ad_sync", "ad_set_acceptance",
    "ad_debug_logits", "ad_debug_encoder_memory", "ad_debug_stage_timeline", "ad_debug_profile_verify", "ad_vocab_argmax_scratch_bytes", "ad_vocab_argmax",
    "ad_vocab_argmax_static", "ad_debug_wait_probe", "ad_debug_grid_barrier_probe",
    "ad_linear",
]


class ModelCfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("d_model", "n_heads", "d_ffn", "vocab", "n_enc", "n_dec", "dtype", "max_batch", "max_src",
                 "max_tgt", "kmax", "bos", "pad", "eos", "mask")] + [("ln_eps", C.c_float), ("has_drafter", C.c_int32)]


class ModelWeights(C.Structure):
    _fields_ = [("matrices", C.c_void_p), ("vectors", C.c_void_p)]


class Weights(C.Structure):
    _fields_ = [("ar", ModelWeights), ("nar", ModelWeights)]


class GenOpts(C.Structure):
    _fields_ = [("mode", C.c_int32), ("k", C.c_int32), ("max_len", C.c_void_p), ("draft_override", C.c_void_p),
                ("override_stride", C.c_int32), ("run_drafter", C.c_int32), ("sync_every", C.c_int32),
                ("use_graph", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("iterations", C.c_int64), ("row_iterations", C.c_int64), ("accepted", C.c_int64),
                ("offered", C.c_int64), ("device_ms", C.c_float), ("encode_ms", C.c_float),
                ("kernel_launches", C.c_int64)]


class AdError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"aggressive_decoding error {code}: {msg}")
        self.code = code


_lib = None


def load():
    """Loads the shared library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with paper_2205_10350_b200.build.build(); "
                          "there is no fallback path")
    lib = C.CDLL(LIB_PATH)
    vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
    sig = {
        "ad_weight_counts": (C.c_int, [C.POINTER(ModelCfg), C.POINTER(sz), C.POINTER(sz)]),
        "ad_query_workspace": (C.c_int, [C.POINTER(ModelCfg), C.POINTER(sz)]),
        "ad_create": (C.c_int, [C.POINTER(ModelCfg), C.POINTER(Weights), vp, sz, vp, C.POINTER(vp)]),
        "ad_destroy": (C.c_int, [vp]),
        "ad_last_error": (C.c_char_p, [vp]),
        "ad_encode": (C.c_int, [vp, vp, i32, vp, i32, i32]),
        "ad_verify_block": (C.c_int, [vp, vp, vp, vp, vp, i32]),
        "ad_commit": (C.c_int, [vp, vp, i32]),
        "ad_force_commit": (C.c_int, [vp, vp, vp, i32]),
        "ad_generate": (C.c_int, [vp, vp, i32, vp, i32, C.POINTER(GenOpts), vp, i32, vp, C.POINTER(Stats), i32]),
        "ad_draft_block": (C.c_int, [vp, i32, vp, vp, i32]),
        "ad_get_state": (C.c_int, [vp, vp, vp, vp]),
        "ad_sync": (C.c_int, [vp]),
        "ad_set_acceptance": (C.c_int, [vp, C.c_int32, C.c_float]),
        "ad_debug_logits": (C.c_int, [vp, i32, vp, sz]),
        "ad_debug_encoder_memory": (C.c_int, [vp, i32, vp, sz]),
        "ad_debug_stage_timeline": (C.c_int, [vp, vp, i32, vp]),
        "ad_debug_profile_verify": (C.c_int, [vp, vp, vp, vp, vp, i32, vp]),
        "ad_vocab_argmax_scratch_bytes": (sz, [i32, i32]),
        "ad_vocab_argmax": (C.c_int, [vp, vp, i32, i32, i32, i32, vp, vp, sz, vp, vp]),
        "ad_vocab_argmax_static": (C.c_int, [vp, vp, i32, i32, i32, i32, vp, vp, vp]),
        "ad_linear": (C.c_int, [vp, vp, vp, i32, i32, i32, i32, vp, vp, vp]),
        "ad_debug_wait_probe": (C.c_int, [vp, i32, vp, vp]),
        "ad_debug_grid_barrier_probe": (C.c_int, [i32, i32, i32, i32, vp, sz, vp, vp, vp]),
    }
    for name, (res, args) in sig.items():
        f = getattr(lib, name)
        f.restype, f.argtypes = res, args
    _lib = lib
    return lib


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def pack_weights(shape, w):
    """Lays one model's tensors out as the header documents: matrices [out, in] in one array, vectors in
    another.  Input convention: ``*.W`` is [in, out]."""
    mats, vecs = [w["emb"]], []
    T = lambda a: np.ascontiguousarray(np.asarray(a).T)
    cat = np.concatenate
    for l in range(shape.n_enc):
        p = f"enc.{l}"
        mats += [cat([T(w[f"{p}.self.{n}.W"]) for n in "qkv"], 0), T(w[f"{p}.self.o.W"]), T(w[f"{p}.ffn1.W"]),
                 T(w[f"{p}.ffn2.W"])]
        vecs += [cat([w[f"{p}.self.{n}.b"] for n in "qkv"]), w[f"{p}.self.o.b"], w[f"{p}.ln1.g"], w[f"{p}.ln1.b"],
                 w[f"{p}.ffn1.b"], w[f"{p}.ffn2.b"], w[f"{p}.ln2.g"], w[f"{p}.ln2.b"]]
    for l in range(shape.n_dec):
        p = f"dec.{l}"
        mats += [cat([T(w[f"{p}.self.{n}.W"]) for n in "qkv"], 0), T(w[f"{p}.self.o.W"]), T(w[f"{p}.cross.q.W"]),
                 cat([T(w[f"{p}.cross.{n}.W"]) for n in "kv"], 0), T(w[f"{p}.cross.o.W"]), T(w[f"{p}.ffn1.W"]),
                 T(w[f"{p}.ffn2.W"])]
        vecs += [cat([w[f"{p}.self.{n}.b"] for n in "qkv"]), w[f"{p}.self.o.b"], w[f"{p}.ln1.g"], w[f"{p}.ln1.b"],
                 w[f"{p}.cross.q.b"], cat([w[f"{p}.cross.{n}.b"] for n in "kv"]), w[f"{p}.cross.o.b"],
                 w[f"{p}.ln2.g"], w[f"{p}.ln2.b"], w[f"{p}.ffn1.b"], w[f"{p}.ffn2.b"], w[f"{p}.ln3.g"], w[f"{p}.ln3.b"]]
    m = cat([np.asarray(a, np.float32).ravel() for a in mats])
    v = cat([np.asarray(a, np.float32).ravel() for a in vecs])
    return m, v


class AggressiveDecoder:
    """One handle of the library: a verifier model (and optionally a drafter) with fixed capacities."""

    def __init__(self, shape, weights, nar_weights=None, max_batch=1, max_src=64, max_tgt=64, kmax=64,
                 bos=0, pad=1, eos=2, mask=3, ln_eps=1e-5, device="cuda:0", stream=None):
        import torch
        self.torch = torch
        self.lib = load()
        self.dev = torch.device(device)
        torch.cuda.set_device(self.dev)
        self.shape = shape
        self.bf16 = shape.dtype == "bf16"
        self.cfg = ModelCfg(shape.d_model, shape.n_heads, shape.d_ffn, shape.vocab, shape.n_enc, shape.n_dec,
                            AD_DTYPE_BF16 if self.bf16 else AD_DTYPE_FP32, max_batch, max_src, max_tgt, kmax,
                            bos, pad, eos, mask, ln_eps, 1 if nar_weights is not None else 0)
        self.max_batch, self.max_src, self.max_tgt, self.kmax = max_batch, max_src, max_tgt, kmax
        nm, nv = C.c_size_t(), C.c_size_t()
        self._check(self.lib.ad_weight_counts(C.byref(self.cfg), C.byref(nm), C.byref(nv)), None)
        self._keep = []
        wstruct = Weights()
        for field, ww in (("ar", weights), ("nar", nar_weights)):
            if ww is None:
                continue
            m, v = pack_weights(shape, ww)
            assert m.size == nm.value and v.size == nv.value, (m.size, nm.value, v.size, nv.value)
            mt = torch.from_numpy(m).to(self.dev)
            if self.bf16:
                mt = mt.to(torch.bfloat16)
            vt = torch.from_numpy(v).to(self.dev)
            self._keep += [mt, vt]
            setattr(wstruct, field, ModelWeights(mt.data_ptr(), vt.data_ptr()))
        nbytes = C.c_size_t()
        self._check(self.lib.ad_query_workspace(C.byref(self.cfg), C.byref(nbytes)), None)
        self.workspace_bytes = nbytes.value
        self.workspace = torch.empty(nbytes.value + 1024, dtype=torch.uint8, device=self.dev)
        base = (self.workspace.data_ptr() + 1023) // 1024 * 1024
        self.stream = stream if stream is not None else torch.cuda.Stream(device=self.dev)
        torch.cuda.synchronize(self.dev)   # weight uploads ran on torch's current stream
        sp = C.c_void_p(self.stream.cuda_stream)
        h = C.c_void_p()
        self._check(self.lib.ad_create(C.byref(self.cfg), C.byref(wstruct), C.c_void_p(base), nbytes.value, sp,
                                       C.byref(h)), None)
        self.h = h
        self.B = 0

    # ------------------------------------------------------------------ helpers
    def _check(self, rc, h):
        if rc != AD_OK:
            msg = self.lib.ad_last_error(h)
            raise AdError(rc, msg.decode() if msg else "")

    def close(self):
        if getattr(self, "h", None):
            self.lib.ad_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ host-array API
    def encode(self, src, src_len):
        src, src_len = _i32(src), _i32(src_len)
        self.B = src.shape[0]
        self._check(self.lib.ad_encode(self.h, src.ctypes.data, src.shape[1], src_len.ctypes.data, self.B, 1), self.h)

    def verify_block(self, drafts, k):
        """drafts [B, <=kmax] (host), k [B].  Returns (argmax [B, kmax], n_accepted [B])."""
        d = np.full((self.B, self.kmax), -1, np.int32)
        drafts = np.asarray(drafts, np.int32)
        d[:, : drafts.shape[1]] = drafts
        k = _i32(k)
        am = np.zeros((self.B, self.kmax), np.int32)
        n = np.zeros(self.B, np.int32)
        self._check(self.lib.ad_verify_block(self.h, d.ctypes.data, k.ctypes.data, am.ctypes.data, n.ctypes.data, 1), self.h)
        return am, n

    def commit(self, n=None):
        if n is None:
            self._check(self.lib.ad_commit(self.h, None, 1), self.h)
        else:
            n = _i32(n)
            self._check(self.lib.ad_commit(self.h, n.ctypes.data, 1), self.h)

    def force_commit(self, tokens, n):
        t = np.full((self.B, self.kmax), -1, np.int32)
        tokens = np.asarray(tokens, np.int32)
        t[:, : tokens.shape[1]] = tokens
        n = _i32(n)
        self._check(self.lib.ad_force_commit(self.h, t.ctypes.data, n.ctypes.data, 1), self.h)

    def draft_block(self, k_cap):
        d = np.zeros((self.B, self.kmax), np.int32)
        k = np.zeros(self.B, np.int32)
        self._check(self.lib.ad_draft_block(self.h, k_cap, d.ctypes.data, k.ctypes.data, 1), self.h)
        return d, k

    def state(self):
        ln, last, fin = (np.zeros(self.B, np.int32) for _ in range(3))
        self._check(self.lib.ad_get_state(self.h, ln.ctypes.data, last.ctypes.data, fin.ctypes.data), self.h)
        return ln, last, fin

    def sync(self):
        self._check(self.lib.ad_sync(self.h), self.h)

    def set_acceptance(self, beta, tau):
        """beta = 0: exact-match verification; beta >= 1: relaxed top-beta / tau verification."""
        self._check(self.lib.ad_set_acceptance(self.h, int(beta), float(tau)), self.h)

    def debug_logits(self, M, which=0):
        t = self.torch.empty((M, self.shape.vocab), dtype=self.torch.float32, device=self.dev)
        self._check(self.lib.ad_debug_logits(self.h, which, C.c_void_p(t.data_ptr()), t.numel()), self.h)
        self.sync()
        return t.cpu().numpy()

    def profile_verify(self, drafts, k, capacity=512):
        """One verification block with every kernel timed on its own: list of (what, microseconds) in launch order."""
        d = np.full((self.B, self.kmax), -1, np.int32)
        drafts = np.asarray(drafts, np.int32)
        d[:, : drafts.shape[1]] = drafts
        k = _i32(k)
        names = C.create_string_buffer(capacity * 64)
        us = np.zeros(capacity, np.float32)
        n = C.c_int32()
        self._check(self.lib.ad_debug_profile_verify(self.h, d.ctypes.data, k.ctypes.data, names, us.ctypes.data, capacity,
                                                     C.byref(n)), self.h)
        raw = names.raw
        return [(raw[i * 64: (i + 1) * 64].split(b"\0")[0].decode(), float(us[i])) for i in range(n.value)]

    def debug_stage_timeline(self):
        """Per-stage (inputs visible, signalled) global-timer stamps of the last persistent decoder pass, in ns."""
        buf = np.zeros(2 * (8 * self.shape.n_dec + 1), np.uint64)
        n = C.c_int32()
        self._check(self.lib.ad_debug_stage_timeline(self.h, buf.ctypes.data, buf.size, C.byref(n)), self.h)
        return buf.reshape(-1, 2)

    def debug_encoder_memory(self, b, src_len):
        t = self.torch.empty((src_len, self.shape.d_model), dtype=self.torch.float32, device=self.dev)
        self._check(self.lib.ad_debug_encoder_memory(self.h, b, C.c_void_p(t.data_ptr()), t.numel()), self.h)
        self.sync()
        return t.cpu().numpy()

    def generate(self, src, src_len, mode="IAD", k=1, max_len=None, draft_override=None, run_drafter=False,
                 sync_every=0, use_graph=True, out=None, out_len=None):
        """Host-array form of ad_generate.  Returns (list of per-row outputs, stats dict)."""
        src, src_len = _i32(src), _i32(src_len)
        B = src.shape[0]
        self.B = B
        opts = GenOpts()
        opts.mode = AD_MODE_GAD if mode == "GAD" else AD_MODE_IAD
        opts.k = k
        keep = []
        if max_len is not None:
            ml = _i32(max_len); keep.append(ml)
            opts.max_len = ml.ctypes.data
        if draft_override is not None:
            ov = _i32(draft_override); keep.append(ov)
            opts.draft_override = ov.ctypes.data
            opts.override_stride = ov.shape[1]
        opts.run_drafter = int(run_drafter)
        opts.sync_every = sync_every
        opts.use_graph = int(use_graph)
        if out is None:
            out = np.zeros((B, self.max_tgt), np.int32)
        if out_len is None:
            out_len = np.zeros(B, np.int32)
        st = Stats()
        self._check(self.lib.ad_generate(self.h, src.ctypes.data, src.shape[1], src_len.ctypes.data, B,
                                         C.byref(opts), out.ctypes.data, out.shape[1], out_len.ctypes.data,
                                         C.byref(st), 1), self.h)
        stats = {f[0]: getattr(st, f[0]) for f in Stats._fields_}
        return [out[b, : out_len[b]].copy() for b in range(B)], stats

    # ------------------------------------------------------------------ device-pointer API (no host copies)
    def generate_device(self, src_t, src_len_t, out_t, out_len_t, mode="IAD", k=1, max_len_t=None,
                        override_t=None, run_drafter=False, sync_every=0, use_graph=True):
        """Same call with every array already resident on the device (torch int32 tensors)."""
        opts = GenOpts()
        opts.mode = AD_MODE_GAD if mode == "GAD" else AD_MODE_IAD
        opts.k = k
        if max_len_t is not None:
            opts.max_len = max_len_t.data_ptr()
        if override_t is not None:
            opts.draft_override = override_t.data_ptr()
            opts.override_stride = override_t.shape[1]
        opts.run_drafter = int(run_drafter)
        opts.sync_every = sync_every
        opts.use_graph = int(use_graph)
        st = Stats()
        B = src_t.shape[0]
        self.B = B
        self._check(self.lib.ad_generate(self.h, C.c_void_p(src_t.data_ptr()), src_t.shape[1],
                                         C.c_void_p(src_len_t.data_ptr()), B, C.byref(opts),
                                         C.c_void_p(out_t.data_ptr()), out_t.shape[1],
                                         C.c_void_p(out_len_t.data_ptr()), C.byref(st), 0), self.h)
        return {f[0]: getattr(st, f[0]) for f in Stats._fields_}

    def verify_block_device(self, drafts_t, k_t, argmax_t, n_t):
        self._check(self.lib.ad_verify_block(self.h, C.c_void_p(drafts_t.data_ptr()), C.c_void_p(k_t.data_ptr()),
                                             C.c_void_p(argmax_t.data_ptr()), C.c_void_p(n_t.data_ptr()), 0), self.h)

    def commit_device(self, n_t=None):
        self._check(self.lib.ad_commit(self.h, C.c_void_p(n_t.data_ptr()) if n_t is not None else None, 0), self.h)


def vocab_argmax(x_t, emb_t, status_t=None):
    """Operator-level call: arg-max of x @ emb^T per row.  x_t [M, d], emb_t [V, d], both float32 or bfloat16."""
    import torch
    lib = load()
    M, d = x_t.shape
    V = emb_t.shape[0]
    dtype = AD_DTYPE_BF16 if x_t.dtype == torch.bfloat16 else AD_DTYPE_FP32
    nbytes = lib.ad_vocab_argmax_scratch_bytes(V, M)
    scratch = torch.empty(nbytes + 256, dtype=torch.uint8, device=x_t.device)
    base = (scratch.data_ptr() + 255) // 256 * 256
    out = torch.empty(M, dtype=torch.int32, device=x_t.device)
    rc = lib.ad_vocab_argmax(C.c_void_p(x_t.data_ptr()), C.c_void_p(emb_t.data_ptr()), dtype, M, d, V,
                             C.c_void_p(out.data_ptr()), C.c_void_p(base), nbytes,
                             C.c_void_p(status_t.data_ptr()) if status_t is not None else None,
                             C.c_void_p(torch.cuda.current_stream().cuda_stream))
    if rc != AD_OK:
        raise AdError(rc, "ad_vocab_argmax")
    torch.cuda.synchronize()
    return out


STATIC_SCRATCH_BYTES = 1 << 20


def vocab_argmax_static(x_t, emb_t, out_t, status_t=None):
    """Projection + arg-max for callers that must not allocate device memory at call time.

    Unlike :func:`vocab_argmax`, nothing is allocated here or inside the library: ``out_t`` (int32, [M]) is
    the caller's, and the scratch is an array built into the library (1 MiB per GPU).  Problems that need
    more are refused with ``AD_ERR_CAPACITY``.  Calls on one GPU share that array, so keep them on one
    stream; make the first call on a device outside any stream capture.  Asynchronous on torch's current
    stream."""
    import torch
    lib = load()
    M, d = x_t.shape
    V = emb_t.shape[0]
    dtype = AD_DTYPE_BF16 if x_t.dtype == torch.bfloat16 else AD_DTYPE_FP32
    rc = lib.ad_vocab_argmax_static(C.c_void_p(x_t.data_ptr()), C.c_void_p(emb_t.data_ptr()), dtype, M, d, V,
                                    C.c_void_p(out_t.data_ptr()),
                                    C.c_void_p(status_t.data_ptr()) if status_t is not None else None,
                                    C.c_void_p(torch.cuda.current_stream().cuda_stream))
    if rc != AD_OK:
        msg = lib.ad_last_error(None)
        raise AdError(rc, msg.decode() if msg else "ad_vocab_argmax_static")
    return out_t


def linear(x_t, W_t, bias_t=None, status_t=None):
    """Operator-level call: y = x W^T + bias in FP32.  x_t [M, K], W_t [N, K]."""
    import torch
    lib = load()
    M, K = x_t.shape
    N = W_t.shape[0]
    dtype = AD_DTYPE_BF16 if x_t.dtype == torch.bfloat16 else AD_DTYPE_FP32
    y = torch.empty((M, N), dtype=torch.float32, device=x_t.device)
    rc = lib.ad_linear(C.c_void_p(x_t.data_ptr()), C.c_void_p(W_t.data_ptr()),
                       C.c_void_p(bias_t.data_ptr()) if bias_t is not None else None, dtype, M, K, N,
                       C.c_void_p(y.data_ptr()), C.c_void_p(status_t.data_ptr()) if status_t is not None else None,
                       C.c_void_p(torch.cuda.current_stream().cuda_stream))
    if rc != AD_OK:
        raise AdError(rc, "ad_linear")
    torch.cuda.synchronize()
    return y
