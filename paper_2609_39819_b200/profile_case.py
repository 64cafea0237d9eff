"""Small, self-terminating cases of one kernel family each, sized for a profiler capture (inputs
larger than L2, a few GB on the device at most, a handful of launches).

    python -m paper_2609_39819_b200.profile_case mover      # paged KV mover, 8B-class blocks, HBM -> HBM
    python -m paper_2609_39819_b200.profile_case mover_toy  # the same with 16 KiB blocks (4 KiB chunks)
    python -m paper_2609_39819_b200.profile_case mover_host # the same blocks, HBM -> pinned host tier and back
    python -m paper_2609_39819_b200.profile_case hash_big   # stand-alone hasher on 64 Mi tokens (256 MiB > L2)
    python -m paper_2609_39819_b200.profile_case exchange   # 1024 blocks each way over the host link: one call vs two
    python -m paper_2609_39819_b200.profile_case lookup     # hash + table lookup of 16 x 16,128-block calls
    python -m paper_2609_39819_b200.profile_case select     # classify + select 10% of 1 Mi resident blocks
    python -m paper_2609_39819_b200.profile_case c4         # the whole metadata stress at full size (C4)
    python -m paper_2609_39819_b200.profile_case mover_remote  # host tier <-> third tier, third tier -> HBM
    python -m paper_2609_39819_b200.profile_case mover_ctas # bandwidth against the number of thread blocks the mover may use
    python -m paper_2609_39819_b200.profile_case overlap    # a GEMM loop beside an offload: what the mover's grid size costs
    python -m paper_2609_39819_b200.profile_case sweep      # C5: movement bandwidth sweep (markdown table)
Each prints one line with CUDA-event timings of its launches.
"""
from __future__ import annotations

import sys

import numpy as np


def _events(torch, fn, n):
    out = []
    for _ in range(n):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); fn(); b.record(); torch.cuda.synchronize()
        out.append(round(a.elapsed_time(b), 4))
    return out


def sweep(torch, B, W):
    """C5: n = 1 .. 65,536 blocks x block sizes x {contiguous, permuted} ids x {gather to the host tier, scatter
    back, HBM -> HBM}; 3 warm-ups, best and median of 10 launches, CUDA events. The pools are capped at 8 GiB
    (HBM) and 4 GiB (pinned host), which caps n for the large blocks."""
    def bench(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(10):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record(); torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        ts.sort()
        return ts[0], ts[len(ts) // 2]

    print("| block | layout | ids | n | gather HBM->host GB/s (best / median) | scatter host->HBM GB/s | HBM->HBM GB/s read+write |")
    print("|---|---|---|---:|---:|---:|---:|")
    for geo in (W.GEO_TOY, W.GEO_128K, W.GEO_512K, W.GEO_8B, W.GEO_GLM):
        n_hbm = min(131072, (8 << 30) // geo.block_bytes)
        n_host = min(65536, (4 << 30) // geo.block_bytes)
        for layout in (0, 1):
            eng = B.Engine(n_hbm_blocks=n_hbm, n_host_blocks=n_host, max_contexts=2, pool_layout=layout, max_tokens=1 << 12,
                           max_messages=64, max_batch_blocks=65536, zero_pools=False, **geo.kwargs())
            n = 1
            while n <= 65536:
                nn = min(n, n_host)
                for perm in (False, True):
                    src = torch.from_numpy(W.ids_c5(1, nn, n_hbm // 2, perm).view(np.int32)).cuda()
                    dst = torch.from_numpy(W.ids_c5(2, nn, n_host, perm).view(np.int32)).cuda()
                    d2 = (torch.from_numpy(W.ids_c5(3, nn, n_hbm // 2, perm).view(np.int32)) + n_hbm // 2).cuda()
                    gb = nn * geo.block_bytes / 1e6
                    g = bench(lambda: eng.copy_blocks(0, src, 1, dst))
                    sc = bench(lambda: eng.copy_blocks(1, dst, 0, src))
                    hh = bench(lambda: eng.copy_blocks(0, src, 0, d2))
                    print(f"| {geo.block_bytes >> 10} KiB | {'layer' if layout == 0 else 'block'}-major | "
                          f"{'permuted' if perm else 'contiguous'} | {nn} | {gb / g[0]:.1f} / {gb / g[1]:.1f} | "
                          f"{gb / sc[0]:.1f} / {gb / sc[1]:.1f} | {2 * gb / hh[0]:.1f} / {2 * gb / hh[1]:.1f} |", flush=True)
                if nn < n:
                    break
                n *= 4
            eng.close()
            del eng
            torch.cuda.empty_cache()


def main(case: str):
    import torch
    from . import binding as B, workloads as W
    torch.cuda.set_device(0)
    if case in ("mover", "mover_toy"):
        geo, n_slots, n = (W.GEO_8B, 1536, 1024) if case == "mover" else (W.GEO_TOY, 196608, 131072)
        eng = B.Engine(n_hbm_blocks=n_slots, n_host_blocks=n_slots, max_contexts=2, max_tokens=1 << 12, max_messages=64,
                       max_batch_blocks=max(n, 4096), host_pool_on_device=True, zero_pools=False, **geo.kwargs())
        src = torch.from_numpy(W.ids_c5(1, n, n_slots, True).view(np.int32)).cuda()
        dst = torch.from_numpy(W.ids_c5(2, n, n_slots, True).view(np.int32)).cuda()
        ms = _events(torch, lambda: eng.copy_blocks(0, src, 1, dst), 3)
        gb = n * geo.block_bytes / 1e9
        print(f"{case}: {n} blocks x {geo.block_bytes} B, permuted ids, ms per launch {ms}, "
              f"read+write GB/s {[round(2 * gb / (m / 1e3), 1) for m in ms]}")
    elif case == "mover_host":
        geo, n_slots, n = W.GEO_8B, 768, 512
        eng = B.Engine(n_hbm_blocks=n_slots, n_host_blocks=n, max_contexts=2, max_tokens=1 << 12, max_messages=64,
                       max_batch_blocks=4096, zero_pools=False, **geo.kwargs())
        src = torch.from_numpy(W.ids_c5(1, n, n_slots, True).view(np.int32)).cuda()
        dst = torch.from_numpy(W.ids_c5(2, n, n, True).view(np.int32)).cuda()
        g = _events(torch, lambda: eng.copy_blocks(0, src, 1, dst), 2)
        sc = _events(torch, lambda: eng.copy_blocks(1, dst, 0, src), 2)
        gb = n * geo.block_bytes / 1e9
        print(f"mover_host: {n} blocks x {geo.block_bytes} B; gather to host ms {g} = {[round(gb / (m / 1e3), 1) for m in g]} GB/s; "
              f"scatter from host ms {sc} = {[round(gb / (m / 1e3), 1) for m in sc]} GB/s")
    elif case == "mover_staged":
        # offload / reload through the staging ring and the copy engines (the default for blocks >= 512 KiB between HBM
        # and a pinned host tier), against the same lists through the kernel that reads / writes host memory itself
        geo, n = W.GEO_8B, 512
        eng = B.Engine(n_hbm_blocks=n, n_host_blocks=n, max_contexts=2, max_tokens=1 << 16, max_messages=64,
                       max_batch_blocks=4096, zero_pools=False, **geo.kwargs())
        rng = np.random.default_rng(3)
        eng.spawn(0)
        eng.append(0, rng.integers(0, W.VOCAB, 16 * n, dtype=np.uint32))
        eng.map_blocks([0], 0); eng.map_blocks([0], 1); eng.prefill_done(0)
        gb = n * geo.block_bytes / 1e9
        for variant, name in ((0, "staging ring + copy engines"), (2, "kernel over mapped host memory")):
            eng.set_mover_variant(variant)
            out = rng.permutation(n).astype(np.uint32)
            for rep in range(2):
                o = _events(torch, lambda: eng.offload(out), 1)
                back = rng.permutation(n).astype(np.uint32)
                r = _events(torch, lambda: eng.reload(back), 1)
                print(f"mover_staged [{name}]: {n} blocks x {geo.block_bytes} B, permuted lists; offload {o[0]:.2f} ms = "
                      f"{gb / (o[0] / 1e3):.1f} GB/s, reload {r[0]:.2f} ms = {gb / (r[0] / 1e3):.1f} GB/s")
    elif case == "mover_remote":
        # host tier <-> the buffer standing in for the remote tier (both pinned host memory): the mover reads over
        # the host link and writes back over it, so both directions of the link carry the payload at once
        geo, n = W.GEO_8B, 512
        eng = B.Engine(n_hbm_blocks=n, n_host_blocks=n, n_remote_blocks=n, max_contexts=2, max_tokens=1 << 12,
                       max_messages=64, max_batch_blocks=4096, zero_pools=False, **geo.kwargs())
        src = torch.from_numpy(W.ids_c5(1, n, n, True).view(np.int32)).cuda()
        dst = torch.from_numpy(W.ids_c5(2, n, n, True).view(np.int32)).cuda()
        down = _events(torch, lambda: eng.copy_blocks(1, src, 2, dst), 2)
        up = _events(torch, lambda: eng.copy_blocks(2, dst, 0, src), 2)
        gb = n * geo.block_bytes / 1e9
        print(f"mover_remote: {n} blocks x {geo.block_bytes} B; host -> remote ms {down} = {[round(gb / (m / 1e3), 1) for m in down]} GB/s; "
              f"remote -> HBM ms {up} = {[round(gb / (m / 1e3), 1) for m in up]} GB/s")
    elif case == "mover_ctas":
        # how many thread blocks a move needs: HBM -> HBM, HBM -> host, host -> HBM against the grid limit
        geo, n = W.GEO_8B, 512
        eng = B.Engine(n_hbm_blocks=2 * n, n_host_blocks=n, max_contexts=2, max_tokens=1 << 12, max_messages=64,
                       max_batch_blocks=4096, zero_pools=False, **geo.kwargs())
        a = torch.from_numpy(W.ids_c5(1, n, n, True).view(np.int32)).cuda()
        b = torch.from_numpy(W.ids_c5(2, n, n, True).view(np.int32)).cuda()
        b2 = b + n
        gb = n * geo.block_bytes / 1e9
        print("| thread blocks (256 threads inside the device, 1024 over the link) | HBM -> HBM GB/s (read + write) | HBM -> host GB/s | host -> HBM GB/s |")
        print("|---:|---:|---:|---:|")
        for ctas in (1, 2, 4, 8, 16, 32, 64, 148, 296, 592, 0):
            eng.set_mover_ctas(ctas)
            dd = min(_events(torch, lambda: eng.copy_blocks(0, a, 0, b2), 3))
            dh = min(_events(torch, lambda: eng.copy_blocks(0, a, 1, b), 2))
            hd = min(_events(torch, lambda: eng.copy_blocks(1, b, 0, a), 2))
            print(f"| {ctas if ctas else 'automatic'} | {2 * gb / (dd / 1e3):.0f} | {gb / (dh / 1e3):.1f} | {gb / (hd / 1e3):.1f} |")
    elif case == "overlap":
        # a dense bf16 GEMM loop on one stream while the mover pushes 2 GiB to the pinned host tier on another:
        # GEMM time alone and beside movers of different grid sizes
        geo, n = W.GEO_8B, 1024
        eng = B.Engine(n_hbm_blocks=n, n_host_blocks=n, max_contexts=2, max_tokens=1 << 12, max_messages=64,
                       max_batch_blocks=4096, zero_pools=False, **geo.kwargs())
        src = torch.from_numpy(W.ids_c5(1, n, n, True).view(np.int32)).cuda()
        dst = torch.from_numpy(W.ids_c5(2, n, n, True).view(np.int32)).cuda()
        x = torch.randn(8192, 8192, dtype=torch.bfloat16, device="cuda")
        y = torch.randn(8192, 8192, dtype=torch.bfloat16, device="cuda")
        s_move, s_gemm = torch.cuda.Stream(), torch.cuda.Stream()
        n_gemm = 40

        def run(ctas):
            torch.cuda.synchronize()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if ctas is not None:
                eng.set_mover_ctas(ctas)
                with torch.cuda.stream(s_move):
                    m0.record(); eng.copy_blocks(0, src, 1, dst); m1.record()
            with torch.cuda.stream(s_gemm):
                g0.record()
                for _ in range(n_gemm):
                    torch.matmul(x, y)
                g1.record()
            torch.cuda.synchronize()
            return g0.elapsed_time(g1), (m0.elapsed_time(m1) if ctas is not None else 0.0)

        run(None); run(0)
        flop = 2 * 8192 ** 3 * n_gemm
        gb = n * geo.block_bytes / 1e9
        cases = [("GEMM alone", None), ("beside the mover, automatic grid (4 blocks of 1024 threads)", 0)] + \
                [(f"beside the mover on {c} blocks of 1024 threads", c) for c in (1, 2, 8, 32, 148, 296)]
        for label, ctas in cases:
            g, m = min(run(ctas) for _ in range(3))
            mv = f", move {m:.1f} ms = {gb / (m / 1e3):.1f} GB/s" if ctas is not None else ""
            print(f"overlap: {label}: {n_gemm} GEMMs in {g:.1f} ms = {flop / (g / 1e3) / 1e12:.0f} TFLOP/s{mv}")
    elif case == "exchange":
        geo, n = W.GEO_8B, (int(sys.argv[2]) if len(sys.argv) > 2 else 1024)    # a smaller n for profiler captures
        eng = B.Engine(n_hbm_blocks=3 * n, n_host_blocks=3 * n, max_contexts=2, max_tokens=1 << 12, max_messages=64,
                       max_batch_blocks=4 * n, zero_pools=False, **geo.kwargs())
        ar = np.arange(n, dtype=np.uint32)
        eng.debug_load_resident(ar + 1000, np.ones(n, np.uint8), ar, ar, ar, 0)            # n idle blocks in HBM
        eng.debug_load_resident(ar + 100000, np.ones(n, np.uint8), ar, ar, ar, 1)          # n idle blocks on the host
        gb = n * geo.block_bytes / 1e9

        def lists():
            return np.nonzero(eng.get_entries(0)["key"])[0], np.nonzero(eng.get_entries(1)["key"])[0]

        res = {"exchange": [], "reload_then_offload": []}
        for rep in range(4):
            for mode in ("exchange", "reload_then_offload"):
                out, inn = lists()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                if mode == "exchange":
                    r = eng.exchange(out, inn)
                else:
                    r = (eng.reload(inn), eng.offload(out))
                b.record(); torch.cuda.synchronize()
                if rep:
                    res[mode].append(round(a.elapsed_time(b), 2))
        # the exchange against the number of thread blocks its mover may use (0 = the library's own choice)
        by_ctas = {}
        for ctas in (2, 4, 8, 16, 32, 64, 148, 0):
            eng.set_mover_ctas(ctas)
            ms = []
            for rep in range(3):
                out, inn = lists()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); eng.exchange(out, inn); b.record(); torch.cuda.synchronize()
                ms.append(a.elapsed_time(b))
            by_ctas[ctas] = round(2 * gb / (min(ms) / 1e3), 1)
        print(f"exchange GB/s (both directions together) by thread blocks: {by_ctas}")
        # reference: the copy engines driving both directions at once (two streams, 2 GiB pinned each way)
        h1 = torch.empty(2 << 30, dtype=torch.uint8, pin_memory=True); d1 = torch.empty(2 << 30, dtype=torch.uint8, device="cuda")
        h2 = torch.empty(2 << 30, dtype=torch.uint8, pin_memory=True); d2 = torch.empty(2 << 30, dtype=torch.uint8, device="cuda")
        s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
        best = 1e9
        for rep in range(5):
            torch.cuda.synchronize()
            t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
            t0.record()
            s1.wait_stream(torch.cuda.current_stream()); s2.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(s1):
                d1.copy_(h1, non_blocking=True)
            with torch.cuda.stream(s2):
                h2.copy_(d2, non_blocking=True)
            torch.cuda.current_stream().wait_stream(s1); torch.cuda.current_stream().wait_stream(s2)
            t1.record(); torch.cuda.synchronize()
            if rep:
                best = min(best, t0.elapsed_time(t1))
        print(f"copy engines, both directions at once: {2 * (2 << 30) / best / 1e6:.1f} GB/s together")
        print(f"exchange: {n} blocks x {geo.block_bytes} B in each direction per call; ms {res}; "
              f"GB/s both directions together { {k: [round(2 * gb / (m / 1e3), 1) for m in v] for k, v in res.items()} }")
    elif case == "hash_big":
        n_tok = 64 << 20
        tok = torch.randint(0, W.VOCAB, (n_tok,), dtype=torch.int32, device="cuda")
        ms = _events(torch, lambda: B.hash_tokens(tok, 0), 8)
        nb = n_tok // 16
        print(f"hash_big: {nb} blocks, ms per call {ms}, blocks/s {[round(nb / (m / 1e3)) for m in ms]}, "
              f"GB/s at 72 B per block {[round(72 * nb / (m / 1e3) / 1e9, 1) for m in ms]}")
    elif case in ("lookup", "select"):
        n_res, n_calls = (1 << 20, 64) if case == "lookup" else (1 << 20, 4)
        inp = W.inputs_c4(1, n_resident=n_res, chain_blocks=16128, n_calls=n_calls)
        eng = B.Engine(n_hbm_blocks=n_res, n_host_blocks=0, max_contexts=n_calls + 1, metadata_only=True,
                       max_tokens=(n_calls + 2) * 16128 * 16 * 2, max_messages=1024, max_batch_blocks=n_calls * 16128,
                       **W.GEO_TOY.kwargs())
        keys = np.concatenate([B.hash_tokens(torch.from_numpy(c.view(np.int32)).cuda()).cpu().numpy().view(np.uint64)
                               for c in inp.chain_tokens])
        eng.debug_load_resident(keys, inp.state, inp.stamp, inp.depth, inp.slot, 0)
        call_tok = [torch.from_numpy(t.view(np.int32)).cuda() for t in inp.calls]

        def fresh_contexts():
            for i, t in enumerate(call_tok):
                eng.spawn(i)
                eng.append(i, t)
        if case == "select":
            fresh_contexts()
        if case == "lookup":
            # both forms of the hash + probe stage, each with a cold L2 (a 512 MiB fill before every batch)
            eng.set_profiling(True)
            flush = torch.empty(1 << 29, dtype=torch.uint8, device="cuda")
            for variant in (1, 2, 1, 2):
                eng.set_lookup_variant(variant)
                ms, kms = [], []
                for rep in range(4):
                    fresh_contexts()          # nothing to resume from: every block is digested
                    flush.fill_(rep)
                    k0 = eng.get_stats()["lookup_ns"]
                    ms += _events(torch, lambda: eng.map_blocks(list(range(n_calls)), 0), 1)
                    kms.append(round((eng.get_stats()["lookup_ns"] - k0) / 1e6, 4))
                    for c in range(n_calls):
                        eng.terminate(c)
                print(f"lookup variant {variant}: {n_calls} calls x 16128 blocks against {n_res} resident, cold L2: "
                      f"ms per batch {ms}, kernels ms {kms}, blocks/s (kernels) {[round(n_calls * 16128 / (m / 1e3)) for m in kms]}")
        else:
            ms = _events(torch, lambda: eng.select_victims(0, n_res // 10), 3)
            print(f"select: {n_res // 10} victims of {n_res} resident, ms per call {ms}")
    elif case == "c4":
        n_res, n_calls = 1 << 20, 64
        inp = W.inputs_c4(1, n_resident=n_res, chain_blocks=16128, n_calls=n_calls)
        eng = B.Engine(n_hbm_blocks=n_res, n_host_blocks=0, max_contexts=n_calls + 1, metadata_only=True,
                       max_tokens=(n_calls + 2) * 16128 * 16 * 2, max_messages=1024, max_batch_blocks=n_calls * 16128,
                       **W.GEO_TOY.kwargs())
        keys = np.concatenate([B.hash_tokens(torch.from_numpy(c.view(np.int32)).cuda()).cpu().numpy().view(np.uint64)
                               for c in inp.chain_tokens])
        eng.debug_load_resident(keys, inp.state, inp.stamp, inp.depth, inp.slot, 0)
        ids = list(range(n_calls))
        for i, t in enumerate(inp.calls):
            eng.spawn(i)
            eng.append(i, torch.from_numpy(t.view(np.int32)).cuda())
        res = {}
        for frac in (0.10, 0.35, 0.75):
            res[f"select_{int(frac * 100)}pct_ms"] = _events(torch, lambda: eng.select_victims(0, int(n_res * frac)), 3)
        res["lookup_batch_ms"] = _events(torch, lambda: eng.map_blocks(ids, 0), 1)
        res["classify_after_lookup_ms"] = _events(torch, lambda: eng.classify(), 1)      # event-driven: the batch's contexts
        eng.set_classify_mode(1)
        res["classify_full_ms"] = _events(torch, lambda: eng.classify(), 2)              # recomputed from zero
        eng.set_classify_mode(0)
        v, _s = eng.select_victims(0, n_res // 10)
        res["drop_10pct_ms"] = _events(torch, lambda: eng.offload(v), 1)
        res["admit_batch_ms"] = _events(torch, lambda: eng.map_blocks(ids, 1), 1)
        st = eng.get_stats()
        print(f"c4: {n_res} resident, {n_calls} calls x 16128 blocks; hits {st['hits_hbm']}, inserted {st['inserted']}, "
              f"adopted {st['adopted']}, tombstones {st['tombstones']}; {res}")
    elif case == "sweep":
        sweep(torch, B, W)
    else:
        raise SystemExit(__doc__)


if __name__ == "__main__":
    main(sys.argv[1] if len(sys.argv) > 1 else "")
