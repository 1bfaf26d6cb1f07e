"""Run ONE op of the library on a chosen shape a few times (CUDA-event timing).

Meant for profiler captures of a single kernel on a small case and for quick shape sweeps:

    python -m paper_2608_00938_b200.opbench linear --M 32768 --N 2048 --K 512 --iters 5
    python -m paper_2608_00938_b200.opbench cross_attn --B 16 --M 2048 --T 1024 --iters 5
    python -m paper_2608_00938_b200.opbench self_attn --B 32 --M 2048 --t 3
    python -m paper_2608_00938_b200.opbench topk --B 32 --M 2048 --V 1024 --K 2048
"""
from __future__ import annotations

import argparse

import torch

from . import api


def _time(fn, iters, warm=2):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    ts = []
    for _ in range(iters):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); fn(); b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b) * 1e3)
    return sorted(ts)[len(ts) // 2]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["linear", "cross_attn", "self_attn", "topk", "mask", "lookup", "layer_norm", "log_softmax", "row_stats"])
    for name, default in (("B", 32), ("M", 2048), ("N", 2048), ("K", 512), ("T", 1024), ("H", 8), ("d", 64),
                          ("V", 1024), ("t", 3), ("iters", 5)):
        ap.add_argument(f"--{name}", type=int, default=default)
    ap.add_argument("--density", type=float, default=0.21, help="mask: fraction of tokens that are catalog children")
    ap.add_argument("--fill", type=float, default=0.43, help="mask: fraction of Bloom bits set")
    ap.add_argument("--matcher", default="bloom", choices=["none", "node", "bloom"])
    ap.add_argument("--f32out", action="store_true")
    ap.add_argument("--residual", action="store_true")
    ap.add_argument("--relu", action="store_true")
    ap.add_argument("--bf16stream", action="store_true", help="linear / layer_norm: bf16 residual stream")
    ap.add_argument("--kway", type=int, default=1, help="lookup: static k-way partitioned rows with this k at every level")
    ap.add_argument("--logits", action="store_true", help="mask: fused log-softmax form (input = logits, in place)")
    ap.add_argument("--allow-only", action="store_true", help="mask: the constraint alone (grace_gtm_allow_bits)")
    ap.add_argument("--allowed", type=float, default=-1.0,
                    help="linear: grace_linear_logits_allowed with this fraction of the columns allowed (folded LayerNorm)")
    ap.add_argument("--inplace", action="store_true",
                    help="self_attn: the cache slabs are the steps' QKV projections (nothing written but the output)")
    ap.add_argument("--folded", action="store_true",
                    help="linear: LayerNorm folded into the epilogue (row pair + column bias; centred rows)")
    a = ap.parse_args()
    dev = "cuda:0"
    torch.manual_seed(0)
    bf = lambda *s: torch.randn(*s, device=dev).to(torch.bfloat16)
    if a.op == "linear":
        x, w = bf(a.M, a.K), bf(a.N, a.K) * 0.05
        y = torch.zeros(a.M, a.N, device=dev, dtype=torch.float32 if (a.f32out or a.residual) and not a.bf16stream
                        else torch.bfloat16)
        if a.allowed >= 0:
            # logits GEMM that stores only the allowed logits (random allow bits of the given density) + partials
            aff, cb = torch.ones(a.M, 2, device=dev), torch.zeros(a.N, device=dev)
            bits = torch.zeros(a.M, a.N // 64, dtype=torch.int64, device=dev)
            for bit in range(64):
                bits |= (torch.rand(a.M, a.N // 64, device=dev) < a.allowed).to(torch.int64) << bit
            y = torch.zeros(a.M, a.N, device=dev)
            part = torch.zeros(a.M, a.N // 256, 2, device=dev)
            us = _time(lambda: api.grace_linear_logits_allowed(x, w, bits, y, part, -1.0, aff, None, cb), a.iters)
        elif a.folded:
            aff, cb = torch.ones(a.M, 2, device=dev), torch.zeros(a.N, device=dev)
            us = _time(lambda: api.grace_linear_folded_ln(x, w, aff, None, cb, y, a.relu), a.iters)
        elif a.bf16stream:
            us = _time(lambda: api.grace_linear_add_bf16(x, w, y), a.iters)
        else:
            us = _time(lambda: api.grace_linear(x, w, y, y if a.residual else None, a.relu), a.iters)
        print(f"linear M={a.M} N={a.N} K={a.K}: {us:.1f} us, {2.0 * a.M * a.N * a.K / us / 1e6:.1f} TFLOP/s")
    elif a.op == "row_stats":
        R = a.B * a.M
        xs = [bf(R, a.K) for _ in range(3)]                # rotated: 3 x R x K x 2 bytes, larger than L2 at R = 65536
        aff = torch.zeros(R, 2, device=dev)
        i = [0]
        def run():
            i[0] += 1
            api.grace_row_stats_bf16(xs[i[0] % 3], aff)
        us = _time(run, a.iters)
        print(f"row_stats R={R} D={a.K}: {us:.1f} us, {R * (a.K * 2 + 8) / us / 1e3:.0f} GB/s")
    elif a.op == "cross_attn":
        q, k, v = bf(a.B * a.M, a.H, a.d), bf(a.B, a.H, a.T, a.d), bf(a.B, a.H, a.T, a.d)
        o = torch.empty_like(q)
        us = _time(lambda: api.grace_cross_attn(q, k, v, o, a.d ** -0.5), a.iters)
        fl = 4.0 * a.B * a.M * a.H * a.d * a.T
        by = 2 * (2 * q.numel() + 2 * k.numel())
        print(f"cross_attn B={a.B} M={a.M} T={a.T}: {us:.1f} us, {fl / us / 1e6:.1f} TFLOP/s, {by / us / 1e3:.0f} GB/s")
    elif a.op == "self_attn":
        R = a.B * a.M
        Lc = a.t + 1
        kc, vc = bf(Lc, R, a.H, a.d), bf(Lc, R, a.H, a.d)
        par = torch.randint(0, a.M, (Lc, R), device=dev, dtype=torch.int32)
        qkv, o = bf(R, 3, a.H, a.d), torch.empty(R, a.H, a.d, device=dev, dtype=torch.bfloat16)
        if a.inplace:
            slabs = bf(Lc, R, 3, a.H, a.d)
            us = _time(lambda: api.grace_self_attn_inplace(slabs, par, [a.M] * Lc, o, a.B, a.t, a.d ** -0.5), a.iters)
        else:
            us = _time(lambda: api.grace_self_attn(qkv, kc, vc, par, [a.M] * Lc, o, a.B, a.t, a.d ** -0.5), a.iters)
        by = R * a.H * a.d * 2 * ((4 if a.inplace else 6) + 2 * a.t)
        print(f"self_attn R={R} T_self={a.t + 1}: {us:.1f} us, {by / us / 1e3:.0f} GB/s (logical bytes)")
    elif a.op == "topk":
        N = a.M * a.V
        cand = torch.randn(a.B, N, device=dev) * 3 - 8
        ws = torch.empty(api.grace_beam_topk_workspace_bytes(a.B, N, a.K), dtype=torch.uint8, device=dev)
        sc = torch.empty(a.B, a.K, device=dev)
        fl = torch.empty(a.B, a.K, device=dev, dtype=torch.int32)
        pa, tk = torch.empty_like(fl), torch.empty_like(fl)
        us = _time(lambda: api.grace_beam_topk(cand, a.K, a.V, sc, fl, pa, tk, ws), a.iters)
        print(f"topk B={a.B} N={N} K={a.K}: {us:.1f} us, {a.B * N * 4 / us / 1e3:.0f} GB/s")
    elif a.op == "mask":
        # synthetic index with the statistics of a trie level: every row has its own node whose child
        # bitmask has `density` of its bits set; the matcher bits are random with the given fill
        R, W = a.B * a.M, a.V // 64
        bits = torch.zeros(R, W, dtype=torch.int64, device=dev)
        for bit in range(64):
            bits |= (torch.rand(R, W, device=dev) < a.density).to(torch.int64) << bit
        base = torch.arange(R, device=dev, dtype=torch.int32) * 8 + 1
        num_nodes = int(R * 8 + a.V + 2)
        trie = api.make_trie(bits, base, a.V, 4, num_nodes)
        if a.matcher == "bloom":
            words = (1 << 22) // 64
            mb = torch.zeros(a.B, words, dtype=torch.int64, device=dev)
            for bit in range(64):
                mb |= (torch.rand(a.B, words, device=dev) < a.fill).to(torch.int64) << bit
            matcher = api.make_matcher(api.MATCH_PREFIX_BLOOM, mb, 22, 4)
        elif a.matcher == "node":
            mb = torch.randint(-2 ** 62, 2 ** 62, (a.B, (num_nodes + 63) // 64), dtype=torch.int64, device=dev)
            matcher = api.make_matcher(api.MATCH_NODE_BITMASK, mb)
        else:
            matcher = api.make_matcher(api.MATCH_NONE)
        logp = torch.log_softmax(torch.randn(R, a.V, device=dev) * 3, dim=1)
        score = -torch.rand(R, device=dev)
        node = torch.arange(R, device=dev, dtype=torch.int32)
        key = torch.randint(1, a.V, (R,), device=dev, dtype=torch.int64)
        cand = torch.empty_like(logp)
        if a.allow_only:
            # the constraint alone (allow bits from the beam state); GRACE_BLOOM_DSMEM=1 in the environment selects the
            # variant that keeps the request's Bloom filter in the shared memory of a four-CTA cluster
            allow = torch.empty(R, W, dtype=torch.int64, device=dev)
            us = _time(lambda: api.grace_gtm_allow_bits(node, key, trie, matcher, allow, a.B, a.M, 1), a.iters)
            print(f"allow_bits[{a.matcher}] R={R} V={a.V} density={a.density}: {us:.1f} us")
            return
        if a.logits:
            lse = torch.empty(R, device=dev)
            us = _time(lambda: api.grace_gtm_mask_logits(logp, lse, score, node, key, trie, matcher, cand, None, a.B, a.M, 1),
                       a.iters)
        else:
            us = _time(lambda: api.grace_gtm_mask(logp, score, node, key, trie, matcher, cand, None, a.B, a.M, 1), a.iters)
        print(f"mask[{a.matcher}{', fused log-softmax' if a.logits else ''}] R={R} V={a.V} density={a.density}: {us:.1f} us, {2 * R * a.V * 4 / us / 1e3:.0f} GB/s "
              f"(dense-form bytes)")
    elif a.op == "lookup":
        # the paper's index form on a synthetic catalog: --N SIDs (thousands), vocabulary --V, depth --t beams
        import numpy as np
        import synth
        rng = synth.rng_for(4, 900)
        n_sids, L, depth = a.N * 1000, 4, a.t
        sids = synth.catalog(rng, n_sids, a.V, L)
        layout = synth.TargetingLayout()
        loc_rows = synth.location_rows(rng, layout)
        ad_sid, ad_bm, ad_bl = synth.ads_for_sids(rng, n_sids, layout, loc_rows)
        ubm, ubl, _ = synth.request_attributes(rng, a.B, layout, loc_rows, n_loc=64)
        if a.kway > 1:
            h = api.grace_gtm_index_build_kway(sids, a.V, ad_sid, ad_bm, ad_bl, k_level=[a.kway] * (L + 1))
        else:
            h = api.grace_gtm_index_build(sids, a.V, ad_sid, ad_bm, ad_bl)
        index = api.make_gtm_index(h, ubm, np.ascontiguousarray(ubl), dev)
        level = np.unique(sids[:, :depth], axis=0)                      # nodes of that depth, in id order
        first = int(api.grace_trie_count_nodes(sids, a.V)[depth])
        pick = rng.integers(0, level.shape[0], size=a.B * a.M)
        node = torch.from_numpy((first + pick).astype(np.int32)).to(dev)
        R = a.B * a.M
        logp = torch.log_softmax(torch.randn(R, a.V, device=dev) * 3, dim=1)
        score = -torch.rand(R, device=dev)
        cand = torch.empty_like(logp)
        allow = torch.zeros(R, a.V // 64, dtype=torch.int64, device=dev)
        us = _time(lambda: api.grace_gtm_lookup(logp, score, node, index, cand, allow, a.B, a.M), a.iters)
        deg = np.diff(h["node_offsets"])[first + pick].mean()
        frac = float((allow != 0).any(dim=1).float().mean())
        kept = float(torch.isfinite(cand).float().sum()) / R
        slots = h["bitmask_index"].shape[0]
        print(f"lookup R={R} V={a.V} depth={depth} k={a.kway}: kept {kept:.1f} of {deg:.1f} children per beam, "
              f"{slots} matcher slots")
        print(f"lookup R={R} V={a.V} depth={depth}: {us:.1f} us, {2 * R * a.V * 4 / us / 1e3:.0f} GB/s (dense-form bytes); "
              f"children/beam {deg:.1f}, rows with a survivor {frac:.2f}, tables {h['bitmask_table'].shape[0]} / "
              f"{h['bloom_table'].shape[0]} unique rows for {h['num_nodes'] - 1} entries")
    elif a.op == "layer_norm":
        R = a.B * a.M
        x = torch.randn(R, a.K, device=dev)
        if a.bf16stream:
            x = x.to(torch.bfloat16)
        g, b = torch.ones(a.K, device=dev), torch.zeros(a.K, device=dev)
        o = torch.empty(R, a.K, device=dev, dtype=torch.bfloat16)
        us = _time(lambda: api.grace_layer_norm(x, g, b, o), a.iters)
        print(f"layer_norm R={R} D={a.K}: {us:.1f} us, {R * a.K * (x.element_size() + 2) / us / 1e3:.0f} GB/s")
    else:
        R = a.B * a.M
        z = torch.randn(R, a.V, device=dev)
        us = _time(lambda: api.grace_log_softmax(z), a.iters)
        print(f"log_softmax R={R} V={a.V}: {us:.1f} us, {R * a.V * 8 / us / 1e3:.0f} GB/s")


if __name__ == "__main__":
    main()
