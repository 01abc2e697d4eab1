"""The C-ABI library loads on a machine without a GPU and exports every symbol the header declares;
host-only entry points (sizes, configuration checks) behave."""
import ctypes as C
import os
import re

import pytest

from paper_2205_10350_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "aggressive_decoding.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ad_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def _cfg(shape, **kw):
    args = dict(max_batch=1, max_src=40, max_tgt=40, kmax=40)
    args.update(kw)
    return binding.ModelCfg(shape.d_model, shape.n_heads, shape.d_ffn, shape.vocab, shape.n_enc, shape.n_dec,
                            1 if shape.dtype == "bf16" else 0, args["max_batch"], args["max_src"], args["max_tgt"],
                            args["kmax"], 0, 1, 2, 3, 1e-5, 0)


def test_weight_counts_match_the_documented_layout(lib):
    for shape in (synth.TINY, synth.BASE):
        cfg = _cfg(shape)
        nm, nv = C.c_size_t(), C.c_size_t()
        assert lib.ad_weight_counts(C.byref(cfg), C.byref(nm), C.byref(nv)) == 0
        d, F, V = shape.d_model, shape.d_ffn, shape.vocab
        mats = V * d + shape.n_enc * (4 * d * d + 2 * d * F) + shape.n_dec * (8 * d * d + 2 * d * F)
        assert nm.value == mats
        w = {n: __import__("numpy").zeros(s, "float32") for n, s in synth.weight_names(shape)}
        m, v = binding.pack_weights(shape, w)
        assert (m.size, v.size) == (nm.value, nv.value)
    # per-verify streamed weights of the base model: 6 (6 d^2 + 2 d F) + V d parameters
    d, F, V = 512, 2048, 32000
    assert 6 * (6 * d * d + 2 * d * F) + V * d == 38_404_096


def test_workspace_query_and_config_checks(lib):
    n = C.c_size_t()
    assert lib.ad_query_workspace(C.byref(_cfg(synth.BASE)), C.byref(n)) == 0
    small = n.value
    assert lib.ad_query_workspace(C.byref(_cfg(synth.BASE, max_batch=32, max_src=64, max_tgt=64, kmax=64)), C.byref(n)) == 0
    assert n.value > small > 0
    bad = _cfg(synth.BASE, kmax=300)
    assert lib.ad_query_workspace(C.byref(bad), C.byref(n)) == binding.AD_ERR_ARG
    assert b"kmax" in lib.ad_last_error(None)
    bad = _cfg(synth.BASE)
    bad.n_heads = 7
    assert lib.ad_query_workspace(C.byref(bad), C.byref(n)) == binding.AD_ERR_ARG
    bad = _cfg(synth.BASE)
    bad.eos = 40000
    assert lib.ad_query_workspace(C.byref(bad), C.byref(n)) == binding.AD_ERR_ARG


def test_struct_layouts():
    assert C.sizeof(binding.ModelCfg) == 17 * 4
    assert C.sizeof(binding.GenOpts) == 40
    assert C.sizeof(binding.Stats) == 48


def test_null_handle_calls_are_rejected(lib):
    assert lib.ad_encode(None, None, 1, None, 1, 1) == binding.AD_ERR_ARG
    assert lib.ad_commit(None, None, 1) == binding.AD_ERR_ARG
    assert lib.ad_destroy(None) == binding.AD_ERR_ARG
