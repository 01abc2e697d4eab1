"""The allocation-free projection + arg-max entry point (collected last on purpose: a run that stops at the
first failure has then already been through every other test).

Some users of this library run where device memory cannot be allocated at call time -- inside another
program's memory pool, or in a latency-critical section where cudaMalloc's implicit synchronisation is not
acceptable.  For them ``ad_vocab_argmax_static`` keeps its scratch in an array that is part of the library
itself.  The test drives it through the C ABI twice in a row (the second call finds the array dirty from the
first and from a different problem size) and requires the same ids as the ordinary entry point, which takes
its scratch from the caller; the ids are also compared with the CPU checker's projection and arg-max directly,
and torch's allocator counters must not move across the calls (nothing is allocated on the caller's behalf)."""
import numpy as np
import pytest
import torch

from oracle import ad_oracle as O
from paper_2205_10350_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _problem(M, d, V, bf16, seed):
    r = np.random.default_rng(seed)
    x = r.standard_normal((M, d)).astype(np.float32)
    E = (r.standard_normal((V, d)) * 0.02).astype(np.float32)
    tx, tE = torch.tensor(x, device=DEV), torch.tensor(E, device=DEV)
    if bf16:
        tx, tE = tx.bfloat16(), tE.bfloat16()
    return tx, tE


def _checker_ids(tx, tE):
    """The CPU checker's linear map + top-2 on the very values the GPU sees (BF16 inputs widened to FP32)."""
    ops = O.Ops("f32")
    logits = ops.linear(tx.float().cpu().numpy(), tE.float().cpu().numpy().T.copy())
    ids, margins = [], []
    for row in logits:
        i1, v1, i2, v2 = ops.top2(row)
        ids.append(i1); margins.append(v1 - v2)
    return np.array(ids), np.array(margins)


@pytest.mark.parametrize("bf16", [True, False])
def test_static_scratch_variant_matches_the_ordinary_entry_point_twice_in_a_row(bf16):
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    # two different problems back to back: the second call inherits the first call's leftovers
    for call, (M, d, V) in enumerate([(40, 512, 32000), (9, 256, 4100)] if bf16 else [(9, 128, 1000), (33, 128, 700)]):
        tx, tE = _problem(M, d, V, bf16, seed=10 + call)
        ref = binding.vocab_argmax(tx, tE, status)                       # caller-provided scratch
        out = torch.full((M,), -7, dtype=torch.int32, device=DEV)       # the caller's output buffers
        out2 = torch.full((M,), -7, dtype=torch.int32, device=DEV)
        torch.cuda.synchronize()
        before = (torch.cuda.memory_allocated(DEV), torch.cuda.memory_reserved(DEV))
        binding.vocab_argmax_static(tx, tE, out, status)
        # and once more on the same problem, straight away
        binding.vocab_argmax_static(tx, tE, out2, status)
        torch.cuda.synchronize()
        assert (torch.cuda.memory_allocated(DEV), torch.cuda.memory_reserved(DEV)) == before, "the call allocated"
        assert torch.equal(out, ref), f"call {call}: ids differ"         # integer result: must be identical
        assert torch.equal(out2, ref)
        # directly against the CPU checker: exact wherever its top-1/top-2 gap is not a rounding matter
        ids, margins = _checker_ids(tx, tE)
        clear = margins > (1e-2 if bf16 else 1e-4)
        assert clear.sum() >= M // 2
        assert np.array_equal(out.cpu().numpy()[clear], ids[clear]), f"call {call}: ids differ from the checker's"
    assert int(status.item()) == 0


def test_static_scratch_variant_accepts_a_problem_that_fills_its_array_exactly():
    M, d, V = 256, 64, 65536                                             # partials: 2 x 512 tiles x 256 rows x 4 B = 1 MiB
    assert binding.load().ad_vocab_argmax_scratch_bytes(V, M) == binding.STATIC_SCRATCH_BYTES
    tx, tE = _problem(M, d, V, True, seed=5)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = torch.full((M,), -7, dtype=torch.int32, device=DEV)
    binding.vocab_argmax_static(tx, tE, out, status)
    torch.cuda.synchronize()
    assert torch.equal(out, binding.vocab_argmax(tx, tE, status)) and int(status.item()) == 0


def test_static_scratch_variant_reports_why_a_shape_is_refused():
    lib = binding.load()
    tx = torch.zeros((4, 96), device=DEV).bfloat16()                     # BF16 needs d % 64 == 0
    tE = torch.zeros((300, 96), device=DEV).bfloat16()
    out = torch.zeros(4, dtype=torch.int32, device=DEV)
    rc = lib.ad_vocab_argmax_static(tx.data_ptr(), tE.data_ptr(), 1, 4, 96, 300, out.data_ptr(), None, None)
    assert rc == binding.AD_ERR_ARG
    assert b"ad_vocab_argmax_static" in lib.ad_last_error(None)


def test_static_scratch_variant_refuses_problems_beyond_its_array():
    lib = binding.load()
    V, M = 200000, 256                                                   # needs ~3.2 MB of partials
    assert lib.ad_vocab_argmax_scratch_bytes(V, M) > binding.STATIC_SCRATCH_BYTES
    tx = torch.zeros((M, 64), device=DEV).bfloat16()
    tE = torch.zeros((8, 64), device=DEV).bfloat16()                     # never read: the size check comes first
    out = torch.zeros(M, dtype=torch.int32, device=DEV)
    rc = lib.ad_vocab_argmax_static(tx.data_ptr(), tE.data_ptr(), 1, M, 64, V, out.data_ptr(), None, None)
    assert rc == binding.AD_ERR_CAPACITY
    assert b"built-in array" in lib.ad_last_error(None)
