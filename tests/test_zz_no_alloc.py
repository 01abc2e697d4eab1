"""The allocation-free projection + arg-max entry point (collected last on purpose: a run that stops at the
first failure has then already been through every other test).

Some users of this library run where device memory cannot be allocated at call time -- inside another
program's memory pool, or in a latency-critical section where cudaMalloc's implicit synchronisation is not
acceptable.  For them ``ad_vocab_argmax_static`` keeps its scratch in an array that is part of the library
itself.  The test drives it through the C ABI twice in a row (the second call finds the array dirty from the
first and from a different problem size) and requires the same ids as the ordinary entry point, which takes
its scratch from the caller."""
import numpy as np
import pytest
import torch

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


@pytest.mark.parametrize("bf16", [True, False])
def test_static_scratch_variant_matches_the_ordinary_entry_point_twice_in_a_row(bf16):
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    # two different problems back to back: the second call inherits the first call's leftovers
    for call, (M, d, V) in enumerate([(40, 512, 32000), (9, 256, 4100)] if bf16 else [(9, 128, 1000), (33, 128, 700)]):
        tx, tE = _problem(M, d, V, bf16, seed=10 + call)
        ref = binding.vocab_argmax(tx, tE, status)                       # caller-provided scratch
        out = torch.full((M,), -7, dtype=torch.int32, device=DEV)       # the caller's output buffer
        binding.vocab_argmax_static(tx, tE, out, status)
        torch.cuda.synchronize()
        assert torch.equal(out, ref), f"call {call}: ids differ"         # integer result: must be identical
        # and once more on the same problem, straight away
        out2 = torch.full((M,), -7, dtype=torch.int32, device=DEV)
        binding.vocab_argmax_static(tx, tE, out2, status)
        torch.cuda.synchronize()
        assert torch.equal(out2, ref)
    assert int(status.item()) == 0


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
