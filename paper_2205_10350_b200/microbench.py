"""Micro-benchmarks of single kernels and of one verification step, for profiling.

  python -m paper_2205_10350_b200.microbench --op vocab  --M 40 --reps 5
  python -m paper_2205_10350_b200.microbench --op linear --M 40 --K 512 --N 2048 --reps 5
  python -m paper_2205_10350_b200.microbench --op verify --model base --batch 1 --k 16 --prefix 16 --src 32 --reps 20
  python -m paper_2205_10350_b200.microbench --op loop   --model base --sentences 4
  python -m paper_2205_10350_b200.microbench --op gridbar

Timed with CUDA events on the launching stream; prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import statistics

import numpy as np
import torch

from . import binding, synth

MODELS = {"tiny": synth.TINY, "base": synth.BASE, "big": synth.BIG, "mini": synth.MINI_BF16,
          "deep12_2": synth.DEEP_ENC, "bart_base": synth.BART_BASE_SIZED}


def _events(stream, fn, reps, flush=None):
    """Device time of fn per call in microseconds: all calls are enqueued, then the stream is synchronised once."""
    evs = []
    with torch.cuda.stream(stream):
        for i in range(reps + 3):
            if flush is not None:
                flush.fill_(i & 0xFF)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            evs.append((a, b))
    stream.synchronize()
    return [a.elapsed_time(b) * 1e3 for a, b in evs[3:]]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", required=True, choices=["vocab", "linear", "verify", "loop", "gridbar"])
    ap.add_argument("--model", default="base")
    ap.add_argument("--M", type=int, default=40)
    ap.add_argument("--K", type=int, default=512)
    ap.add_argument("--N", type=int, default=2048)
    ap.add_argument("--V", type=int, default=32000)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--k", type=int, default=16)
    ap.add_argument("--prefix", type=int, default=16)
    ap.add_argument("--src", type=int, default=32)
    ap.add_argument("--sentences", type=int, default=4)
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--cold", action="store_true", help="flush L2 (256 MB write) before every timed call")
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    stream = torch.cuda.Stream()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if args.cold else None
    lib = binding.load()
    import ctypes as C
    out = dict(op=args.op, cold=args.cold)

    if args.op == "gridbar":
        scratch = torch.zeros(8192, dtype=torch.uint8, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        result = torch.zeros(4, dtype=torch.float32, device=dev)
        res = {}
        rounds = args.reps * 50
        # variants (negative rounds = -(rounds * 4 + v)): v bit 0 = relaxed polls + one fence, bit 1 = barrier without payload
        names = {0: "acquire_polls_with_payload", 1: "relaxed_polls_with_payload", 2: "acquire_polls_barrier_only", 3: "relaxed_polls_barrier_only"}
        for v, name in names.items():
            res[name] = {}
            for n in (0, 128, 64, 16, 2):
                for _ in range(2):
                    assert lib.ad_debug_grid_barrier_probe(n, -(rounds * 4 + v), -1, 20000, scratch.data_ptr(), scratch.numel(),
                                                           status.data_ptr(), result.data_ptr(), stream.cuda_stream) == 0
                    stream.synchronize()
                res[name][str(n or "all")] = round(float(result[0].item()), 1)
        out.update(ns_per_barrier_by_variant_and_ctas=res, status=int(status.item()))
    elif args.op in ("vocab", "linear"):
        M, K = args.M, args.K
        N = args.V if args.op == "vocab" else args.N
        x = torch.randn((M, K), device=dev).bfloat16()
        W = (torch.randn((N, K), device=dev) * 0.02).bfloat16()
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        if args.op == "vocab":
            nb = lib.ad_vocab_argmax_scratch_bytes(N, M)
            scratch = torch.empty(nb + 256, dtype=torch.uint8, device=dev)
            base = (scratch.data_ptr() + 255) // 256 * 256
            am = torch.empty(M, dtype=torch.int32, device=dev)

            def fn():      # the projection kernel alone (null result pointer: its per-tile partials stay in scratch)
                assert lib.ad_vocab_argmax(x.data_ptr(), W.data_ptr(), 1, M, K, N, None, base, nb,
                                           status.data_ptr(), stream.cuda_stream) == 0
        else:
            y = torch.empty((M, N), dtype=torch.float32, device=dev)

            def fn():
                assert lib.ad_linear(x.data_ptr(), W.data_ptr(), None, 1, M, K, N, y.data_ptr(), status.data_ptr(),
                                     stream.cuda_stream) == 0
        torch.cuda.synchronize()
        ts = _events(stream, fn, args.reps, flush)
        bytes_ = N * K * 2 + M * K * 2
        out.update(M=M, K=K, N=N, us_mean=statistics.mean(ts), us_min=min(ts), weight_bytes=N * K * 2,
                   gbs=bytes_ / (statistics.mean(ts) * 1e-6) / 1e9, status=int(status.item()))
    else:
        shape = MODELS[args.model]
        B = args.batch
        w = synth.make_weights(shape, 0)
        max_tgt = max(args.prefix + args.k, 8)
        dec = binding.AggressiveDecoder(shape, w, max_batch=B, max_src=args.src, max_tgt=max_tgt, kmax=args.k)
        stream = dec.stream
        r = np.random.default_rng(0)
        src = r.integers(4, shape.vocab, size=(B, args.src)).astype(np.int32)
        lens = np.full(B, args.src, np.int32)
        if args.op == "verify":
            dec.encode(src, lens)
            if args.prefix > 0:      # build a committed prefix by teacher forcing
                left = args.prefix
                while left > 0:
                    n = min(left, args.k)
                    toks = r.integers(4, shape.vocab, size=(B, args.k)).astype(np.int32)
                    dec.verify_block(toks, np.full(B, n, np.int32))
                    dec.force_commit(toks, np.full(B, n, np.int32))
                    left -= n
            d_t = torch.tensor(r.integers(4, shape.vocab, size=(B, args.k)).astype(np.int32), device=dev)
            k_t = torch.full((B,), args.k, dtype=torch.int32, device=dev)
            am_t = torch.zeros((B, args.k), dtype=torch.int32, device=dev)
            n_t = torch.zeros(B, dtype=torch.int32, device=dev)
            z_t = torch.zeros(B, dtype=torch.int32, device=dev)

            def fn():
                dec.verify_block_device(d_t, k_t, am_t, n_t)
                dec.commit_device(z_t)           # n = 0: discard, so that every repetition sees the same prefix

            torch.cuda.synchronize()
            ts = _events(stream, fn, args.reps, flush)
            dec.sync()
            out.update(model=args.model, batch=B, k=args.k, prefix=args.prefix, src=args.src,
                       us_mean=statistics.mean(ts), us_min=min(ts), launch="direct (no graph)")
            import os
            if os.environ.get("AD_MEGA") == "1" and os.environ.get("AD_MEGA_TIMELINE") == "1":
                # persistent decoder pass: per stage (inputs visible, signalled) stamps of CTA 0, last step
                tl = dec.debug_stage_timeline().astype(np.int64)
                t0 = int(tl[0, 0])
                out["stage_ready_us"] = [round(1e-3 * (int(a) - t0), 2) for a, _ in tl]
                out["stage_busy_us"] = [round(1e-3 * (int(b) - int(a)), 2) for a, b in tl]
        else:
            tot_it, tot_ms, tot_tok, launches = 0, 0.0, 0, 0
            for s in range(args.sentences):
                g, _ = dec.generate(src, lens, mode="IAD", k=1, max_len=np.full(B, max_tgt, np.int32))
                gg = np.full((B, max_tgt), synth.PAD, np.int32)
                for b in range(B):
                    gg[b, : len(g[b])] = g[b]
                stream_ids = synth.corrupt_stream(gg, [len(x) for x in g], 0.9, shape.vocab, 77, s)
                _, st = dec.generate(src, lens, mode="IAD", k=args.k, max_len=np.full(B, max_tgt, np.int32),
                                     draft_override=stream_ids)
                tot_it += st["iterations"]; tot_ms += st["device_ms"]; tot_tok += st["accepted"]
                launches += st["kernel_launches"]
            out.update(model=args.model, batch=B, k=args.k, iterations=tot_it, tokens=tot_tok,
                       us_per_iteration=1e3 * tot_ms / max(1, tot_it), kernel_launches=launches)
    print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
