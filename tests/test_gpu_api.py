"""Edge cases and error behaviour of the C ABI on the device (no faults: every bad input is turned into an
error code by the host or by the kernels' own checks)."""
import numpy as np
import pytest

from oracle import ad_oracle as O
from paper_2205_10350_b200 import binding, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def setup():
    shape = synth.ModelShape("edge", 64, 2, 128, 50, 1, 1, "fp32")
    w = synth.make_weights(shape, 0, std=0.1)
    dec = binding.AggressiveDecoder(shape, w, max_batch=4, max_src=10, max_tgt=12, kmax=6)
    om = O.Model(shape, w, max_pos=16)
    return dec, om


def test_call_order_and_capacity_errors(setup):
    dec, om = setup
    fresh = binding.AggressiveDecoder(dec.shape, synth.make_weights(dec.shape, 0, std=0.1), max_batch=2, max_src=10,
                                      max_tgt=12, kmax=6)
    fresh.B = 1
    with pytest.raises(binding.AdError) as e:
        fresh.verify_block(np.zeros((1, 6), np.int32), [1])
    assert e.value.code == binding.AD_ERR_STATE
    with pytest.raises(binding.AdError) as e:
        fresh.encode(np.full((3, 10), 5, np.int32), [3, 3, 3])
    assert e.value.code == binding.AD_ERR_CAPACITY
    with pytest.raises(binding.AdError) as e:
        fresh.encode(np.full((1, 10), 5, np.int32), [11])
    assert e.value.code == binding.AD_ERR_CAPACITY
    with pytest.raises(binding.AdError) as e:
        fresh.encode(np.full((1, 10), 5, np.int32), [0])
    assert e.value.code == binding.AD_ERR_ARG
    with pytest.raises(binding.AdError) as e:
        fresh.generate(np.full((1, 10), 5, np.int32), [4], mode="GAD", k=2, run_drafter=True)
    assert e.value.code == binding.AD_ERR_STATE
    with pytest.raises(binding.AdError) as e:
        fresh.generate(np.full((1, 10), 5, np.int32), [4], mode="IAD", k=7)
    assert e.value.code == binding.AD_ERR_ARG


def test_idle_rows_ragged_blocks_commit_and_rollback(setup):
    dec, om = setup
    src = np.array([[5, 6, 7, 8, 9, 10, 11, 12, 13, 14]] * 3, np.int32)
    lens = np.array([10, 4, 7], np.int32)
    dec.encode(src, lens)
    states = [om.state(src[b, : lens[b]], cap=12) for b in range(3)]
    drafts = np.array([[20, 21, 22, 23, 24, 25], [30, -1, -1, -1, -1, -1], [0] * 6], np.int32)
    ks = np.array([6, 1, 0], np.int32)                      # full block, single step, idle row
    am, n = dec.verify_block(drafts, ks)
    assert n[2] == 0
    for b in (0, 1):
        res = states[b].verify_block(0, drafts[b, : ks[b]])
        assert np.array_equal(am[b, : ks[b]], res["pred"]) and n[b] == res["n"]
    # committing more than was accepted is refused and leaves the row alone
    with pytest.raises(binding.AdError) as e:
        dec.commit([int(n[0]) + 1, 0, 0])
    assert e.value.code == binding.AD_ERR_ARG
    ln, last, fin = dec.state()
    assert (ln == 0).all()
    am, n = dec.verify_block(drafts, ks)
    dec.commit()                                             # NULL = commit what was accepted
    ln, last, fin = dec.state()
    assert ln[0] == n[0] and ln[1] == n[1] and ln[2] == 0
    assert last[0] == am[0, n[0] - 1]
    # commit without a fresh verification is a no-op
    dec.commit()
    ln2, _, _ = dec.state()
    assert np.array_equal(ln, ln2)
    # rollback by one and re-verify: same prediction as before at that position
    if ln[0] >= 1:
        dec.commit([-1, 0, 0])
        ln3, last3, _ = dec.state()
        assert ln3[0] == ln[0] - 1
    with pytest.raises(binding.AdError):
        dec.commit([-50, 0, 0])                              # cannot roll back more than was committed
    # k beyond the cache capacity is refused by the device-side check
    with pytest.raises(binding.AdError) as e:
        dec.verify_block(drafts, [7, 0, 0])
    assert e.value.code == binding.AD_ERR_ARG


def test_maximum_sizes_and_cap_reached(setup):
    dec, om = setup
    src = np.full((4, 10), 6, np.int32)
    src[:, ::2] = 9
    lens = np.array([10, 10, 1, 10], np.int32)
    outs, stats = dec.generate(src, lens, mode="IAD", k=6, max_len=[12, 1, 12, 5])
    for b, cap in enumerate([12, 1, 12, 5]):
        g, _ = om.state(src[b, : lens[b]], cap=12).greedy(cap)
        assert np.array_equal(outs[b], g)
    ln, _, fin = dec.state()
    assert (fin == 1).all()


def test_teacher_forcing_rejects_inconsistent_tokens(setup):
    dec, om = setup
    src = np.full((1, 10), 6, np.int32)
    dec.encode(src, [5])
    dec.verify_block(np.array([[20, 21, 22, -1, -1, -1]], np.int32), [3])
    with pytest.raises(binding.AdError) as e:
        dec.force_commit(np.array([[20, 33, 40]], np.int32), [3])     # second token was not what the block fed
    assert e.value.code == binding.AD_ERR_ARG
    dec.verify_block(np.array([[20, 21, 22, -1, -1, -1]], np.int32), [3])
    dec.force_commit(np.array([[20, 21, 40]], np.int32), [3])
    ln, last, _ = dec.state()
    assert ln[0] == 3 and last[0] == 40


def test_bounded_wait_runs_out_and_reports_timeout():
    """A wait on a barrier that nothing completes must give up after its time budget, latch AD_ERR_TIMEOUT and
    leave the GPU usable (no trap, no hang)."""
    import torch
    lib = binding.load()
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    waited = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    assert lib.ad_debug_wait_probe(status.data_ptr(), 300, waited.data_ptr(), None) == binding.AD_OK
    torch.cuda.synchronize()
    assert int(status.item()) == binding.AD_ERR_TIMEOUT
    assert 300 <= int(waited.item()) < 20000, int(waited.item())      # gave up after the budget, not after seconds
    # the context still works afterwards
    x = torch.ones((4, 64), device="cuda:0").bfloat16()
    y = binding.linear(x, x)
    assert float(y[0, 0]) == 64.0


def test_results_are_bit_reproducible_and_independent_of_the_block_partition():
    """Same inputs -> same bits (no floating-point atomics anywhere); and the scores of a position do not depend
    on how many other positions share its block (Eq. 1): one block of 6 equals six single steps."""
    shape = synth.MINI_BF16
    w = synth.make_weights(shape, 0)
    dec = binding.AggressiveDecoder(shape, w, max_batch=2, max_src=12, max_tgt=16, kmax=8)
    r = np.random.default_rng(3)
    src = r.integers(4, shape.vocab, size=(2, 12)).astype(np.int32)
    lens = np.array([12, 7], np.int32)
    toks = r.integers(4, shape.vocab, size=(2, 8)).astype(np.int32)
    runs = []
    for _ in range(2):
        dec.encode(src, lens)
        dec.verify_block(toks, [6, 6])
        runs.append(dec.debug_logits(12))
    assert np.array_equal(runs[0], runs[1])
    dec.encode(src, lens)
    single = []
    for i in range(6):
        step = np.full((2, 8), -1, np.int32)
        step[:, 0] = toks[:, i]
        dec.verify_block(step, [1, 1])
        single.append(dec.debug_logits(2))
        dec.force_commit(step, [1, 1])
    single = np.stack(single)                      # [6, 2, V]
    block = runs[0].reshape(2, 6, -1)              # rows packed row-major
    for b in range(2):
        assert np.abs(block[b] - single[:, b]).max() < 1e-5


def test_encoders_on_two_streams_equal_encoders_in_sequence(monkeypatch):
    """The drafter's encoder runs on a side stream next to the verifier's.  The same handle configuration with the
    two passes in sequence on one stream (AD_NO_CONCURRENT_ENCODERS=1, read when the handle is created) must give the
    same drafts, the same verified tokens and the same encoder memory, bit for bit."""
    shape = synth.MINI_BF16
    w, wn = synth.make_weights(shape, 0), synth.make_weights(shape, 1)
    r = np.random.default_rng(41)
    src = r.integers(4, shape.vocab, size=(3, 14)).astype(np.int32)
    lens = np.array([14, 9, 11], np.int32)
    got = []
    for sequential in (False, True):
        if sequential:
            monkeypatch.setenv("AD_NO_CONCURRENT_ENCODERS", "1")
        dec = binding.AggressiveDecoder(shape, w, wn, max_batch=3, max_src=14, max_tgt=16, kmax=6)
        res = []
        for _ in range(2):                      # second call replays the captured encode graph
            dec.encode(src, lens)
            mem = dec.debug_encoder_memory(1, int(lens[1]))
            drafts, k = dec.draft_block(6)
            ids, n = dec.verify_block(drafts, k)
            res.append((mem, drafts, k, ids, n))
        outs, _ = dec.generate(src, lens, mode="GAD", k=6, max_len=[12, 12, 12], run_drafter=True)
        got.append((res, outs))
        dec.close()
    for (a, b) in zip(got[0][0], got[1][0]):
        for x, y in zip(a, b):
            assert np.array_equal(x, y)
    for x, y in zip(got[0][1], got[1][1]):
        assert np.array_equal(x, y)


def test_token_ids_and_device_side_lengths_outside_their_range_become_error_codes(setup):
    """Ids index the embedding matrix, so every id a caller can supply is range-checked on the device before use:
    the bad id is replaced by [PAD] (sources, fed tokens) or by a slot that matches nothing (drafts), AD_ERR_ARG is
    reported by the next synchronising call, and only valid memory is ever read."""
    import torch
    dec, om = setup
    V = dec.shape.vocab
    good = np.array([[5, 6, 7, 8, 9, 10, 11, 12, 13, 14]], np.int32)
    for bad_id in (V, V + 1000, -3):
        src = good.copy()
        src[0, 2] = bad_id
        with pytest.raises(binding.AdError) as e:
            dec.encode(src, [6])
        assert e.value.code == binding.AD_ERR_ARG
    dec.encode(good, [6])                                   # the handle is usable afterwards
    st = om.state(good[0, :6], cap=12)
    # a draft beyond the vocabulary: reported, and treated as a slot that matches nothing
    drafts = np.array([[20, V, 22, 23, -1, -1]], np.int32)
    with pytest.raises(binding.AdError) as e:
        dec.verify_block(drafts, [4])
    assert e.value.code == binding.AD_ERR_ARG
    # forced tokens beyond the vocabulary are refused, the row stays where it was
    am, n = dec.verify_block(np.array([[20, 21, 22, -1, -1, -1]], np.int32), [3])
    with pytest.raises(binding.AdError) as e:
        dec.force_commit(np.array([[20, 21, V + 5, -1, -1, -1]], np.int32), [3])
    assert e.value.code == binding.AD_ERR_ARG
    assert dec.state()[0][0] == 0
    # device-resident source lengths cannot be seen by the host: max_src + 1 and 0 are clamped and reported
    for bad_len in (dec.max_src + 1, 0, -4):
        t_src = torch.tensor(good, device="cuda:0")
        t_len = torch.tensor([bad_len], dtype=torch.int32, device="cuda:0")
        rc = dec.lib.ad_encode(dec.h, t_src.data_ptr(), 10, t_len.data_ptr(), 1, 0)
        assert rc == binding.AD_OK                            # asynchronous call: the check runs on the device
        with pytest.raises(binding.AdError) as e:
            dec.sync()
        assert e.value.code == binding.AD_ERR_ARG
    dec.encode(good, [6])
    am, n = dec.verify_block(np.array([[20, 21, 22, -1, -1, -1]], np.int32), [3])
    res = st.verify_block(0, np.array([20, 21, 22], np.int32))
    assert np.array_equal(am[0, :3], res["pred"]) and n[0] == res["n"]


def test_grid_barrier_passes_data_and_its_bounded_wait_runs_out():
    """The grid-wide barrier of the persistent kernel: (a) 200 rounds over one CTA per SM, every CTA checking its
    neighbour's word after each barrier; (b) one CTA that never arrives: the others give up after the time budget,
    report AD_ERR_TIMEOUT and return, and the context stays usable."""
    import torch
    lib = binding.load()
    scratch = torch.zeros(8192, dtype=torch.uint8, device="cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    result = torch.zeros(4, dtype=torch.float32, device="cuda:0")
    rc = lib.ad_debug_grid_barrier_probe(0, 200, -1, 20000, scratch.data_ptr(), scratch.numel(), status.data_ptr(),
                                         result.data_ptr(), None)
    assert rc == binding.AD_OK, lib.ad_last_error(None)
    torch.cuda.synchronize()
    r = result.cpu().numpy()
    assert int(status.item()) == 0 and r[1] == 200 and r[2] == 0
    assert 100.0 < r[0] < 20000.0, r[0]                     # nanoseconds per barrier: sub-microsecond to a few microseconds
    print(f"grid barrier over all SMs: {r[0]:.0f} ns per barrier")
    rc = lib.ad_debug_grid_barrier_probe(0, 5, 3, 500, scratch.data_ptr(), scratch.numel(), status.data_ptr(),
                                         result.data_ptr(), None)
    assert rc == binding.AD_OK
    torch.cuda.synchronize()
    assert int(status.item()) == binding.AD_ERR_TIMEOUT and result.cpu().numpy()[1] == 0
    x = torch.ones((4, 64), device="cuda:0").bfloat16()
    assert float(binding.linear(x, x)[0, 0]) == 64.0


def test_per_kernel_profile_of_a_block_changes_nothing(setup):
    """ad_debug_profile_verify: the block is verified as usual (same ids and accepted length as ad_verify_block), and every
    launch comes back with a name and a positive device time."""
    dec, om = setup
    src = np.array([[5, 6, 7, 8, 9, 10, 11, 12, 13, 14]], np.int32)
    dec.encode(src, [10])
    drafts = np.array([[20, 21, 22, 23, 24, 25]], np.int32)
    ids, n = dec.verify_block(drafts, [6])
    prof = dec.profile_verify(drafts, [6])
    ids2, n2 = dec.verify_block(drafts, [6])
    assert np.array_equal(ids, ids2) and n[0] == n2[0]
    names = [p[0] for p in prof]
    assert len(prof) >= 10 and all(us > 0 for _, us in prof)
    assert names[0] == "prepare_verify" and "embed" in names and any(x.startswith("gemm_") for x in names)
    assert names[-1] in ("argmax_accept", "ad_verify_block")
