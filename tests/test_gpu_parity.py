"""CUDA path against the CPU checker, through the C ABI, element by element on seeded inputs.

Bars: index sets, references, centres and counts bit-exact, except where the checker's own margin
to the k-th score or to the similarity threshold is below 1e-4 relative (those positions are counted
and the remaining structure must still be exactly what the checker derives from the GPU's decision);
magnitudes 2e-6 relative; scores 1e-4 relative; kept rows exact copies; CodeBook vectors 1e-5 (fp32)
or 1e-2 (bf16).
"""
import numpy as np
import pytest
import torch

from oracle import spindlekv_oracle as O
from paper_2507_06517_b200 import synth

from gpu_util import (REL_MARGIN, check_codebook_unit, check_evict_unit, generate, make_config, stack_layers, tok_base,
                      torch_dtype, unit_rows, value_tol)

pytestmark = pytest.mark.gpu


def _pass(wl, **kw):
    from paper_2507_06517_b200.pipeline import SpindleKVPass
    return SpindleKVPass(make_config(wl, **kw.pop("cfg", {})), wl.seq_lens, torch_dtype(wl), **kw)


def run_and_check(wl, cfg_kw=None):
    """Runs every layer of ``wl`` and checks every unit.  Returns margin counters."""
    cfg_kw = cfg_kw or {}
    host = generate(wl)
    p = _pass(wl, cfg=cfg_kw, keep_adjacency=True)
    ns, H = wl.n_shallow, wl.n_kv_heads
    stats = {"topk_margin": 0, "adj_margin": 0, "units": 0}
    deep = list(range(ns, wl.n_layers))
    shallow = list(range(ns))
    if deep:
        K = stack_layers(wl, host, deep, "K")
        V = stack_layers(wl, host, deep, "V")
        Q = stack_layers(wl, host, deep, "Q")
        p.evict(K, V, Q)
        assert p.device_status()["evict"][0] == 0
        scores = p.scores.cpu().numpy()
        keep = p.keep_idx.cpu().numpy()
        cnt = p.keep_cnt.cpu().numpy()
        Kk = p.K_kept.float().cpu().numpy()
        Vk = p.V_kept.float().cpu().numpy()
        _, _, k_plan = O.plan_layers(wl.n_layers, ns, wl.seq_lens, wl.window, wl.beta,
                                     reserve_ratio=wl.budget_frac, budget_tokens=wl.budget_tokens)
        assert np.array_equal(k_plan, p.k_ctx_host)
        for li, lam in enumerate(deep):
            for s, l in enumerate(wl.seq_lens):
                tb = tok_base(wl, s)
                Ks = np.stack([unit_rows(wl, host[lam][0], s, j) for j in range(H)])
                Vs = np.stack([unit_rows(wl, host[lam][1], s, j) for j in range(H)])
                k_ctx = int(k_plan[lam, s])
                stats["topk_margin"] += check_evict_unit(
                    wl, host[lam][2][s], Ks, k_ctx, scores[li, :, tb:tb + l], keep[li, :, tb:tb + l], cnt[li, s],
                    score_norm=cfg_kw.get("score_norm", 0))
                for j in range(H):
                    kg = keep[li, j, tb:tb + k_ctx + wl.window]
                    got_k = unit_rows(wl, Kk[li], s, j)[: kg.size]
                    got_v = unit_rows(wl, Vk[li], s, j)[: kg.size]
                    assert np.array_equal(got_k, Ks[j][kg]) and np.array_equal(got_v, Vs[j][kg])
                    stats["units"] += 1
    if shallow:
        for which, idx, theta in (("K", 0, wl.theta_k), ("V", 1, wl.theta_v)):
            G = stack_layers(wl, host, shallow, which)
            p.codebook(G, which)
            st = p.device_status()["codebook"]
            assert st[0] == 0 and st[1][1] == 0
            out = {k: v.float().cpu().numpy() if k == "C" else v.cpu().numpy() for k, v in p.cb[which].items()}
            adj = p.adj.cpu().numpy()
            for li, lam in enumerate(shallow):
                for s, l in enumerate(wl.seq_lens):
                    tb = tok_base(wl, s)
                    for j in range(H):
                        unit = (li * wl.batch + s) * H + j
                        gamma = unit_rows(wl, host[lam][idx], s, j)
                        stats["adj_margin"] += check_codebook_unit(
                            gamma, theta, adj[unit], out["mag"][li, j, tb:tb + l], out["ref"][li, j, tb:tb + l],
                            out["centre_idx"][li, j, tb:tb + l], int(out["n_entries"][li, s, j]),
                            unit_rows(wl, out["C"][li], s, j), value_tol(wl))
                        stats["units"] += 1
    return stats


def test_tiny_fp32_config():
    stats = run_and_check(synth.workload("C1"))
    assert stats["units"] == 2 + 4


def test_ragged_bf16_d128():
    wl = synth.Workload("ragged", 2, 1, 8, 2, 128, "bf16", 32, (1000,), 40, (0.05, 0.3), 4, "recency",
                        budget_tokens=200.0, seed=11)
    run_and_check(wl)


def test_packed_varlen_bf16_d64_pyramid():
    wl = synth.Workload("packed", 3, 1, 4, 2, 64, "bf16", 16, (300, 777, 512), 24, (0.05, 0.3), 2, "recency",
                        budget_frac=0.2, seed=12)
    run_and_check(wl)


def test_mha_fp32_d128_two_sequences():
    wl = synth.Workload("mha", 2, 1, 2, 2, 128, "f32", 32, (200, 200), 10, 0.15, 2, "gauss",
                        budget_tokens=100.0, seed=13)
    run_and_check(wl)


def test_dense_and_sparse_rows_mixed():
    # three big clusters (rows with far more than 32 neighbours use their bit row) next to
    # noisy tokens with few or no neighbours (rows that use neighbour lists)
    wl = synth.Workload("dense", 1, 1, 2, 2, 64, "bf16", 8, (700,), 3, (0.02, 0.6), 2, "gauss",
                        budget_tokens=700.0, seed=17)
    run_and_check(wl)
    wl = synth.Workload("dense32", 1, 1, 2, 2, 128, "f32", 8, (520,), 12, (0.05, 0.2), 2, "gauss",
                        budget_tokens=520.0, seed=18)
    run_and_check(wl)


def test_window_scores_on_tensor_cores_shapes():
    # evicting layers only; every case takes the tensor-core window-score path (bf16, window divides 128)
    cases = [
        # 256 query rows per KV head (two 128-row blocks): 4 x 64 and 8 x 32; several tiles and a ragged tail
        synth.Workload("qb2_w64", 2, 0, 8, 2, 128, "bf16", 64, (1100,), 30, (0.05, 0.3), 4, "recency",
                       budget_tokens=300.0, seed=31),
        synth.Workload("qb2_h8", 1, 0, 16, 2, 64, "bf16", 32, (700,), 30, (0.05, 0.3), 4, "recency",
                       budget_tokens=200.0, seed=32),
        # 192 rows: the second block is half padding; head_dim 64, window 16
        synth.Workload("rows192", 1, 0, 12, 2, 128, "bf16", 32, (515,), 20, 0.2, 2, "gauss",
                       budget_tokens=150.0, seed=33),
        synth.Workload("d64_w16", 2, 0, 16, 4, 64, "bf16", 16, (640,), 20, 0.2, 2, "recency",
                       budget_tokens=100.0, seed=34),
        # fewer rows than one block (rows of the next group's heads are loaded and ignored); window 128
        synth.Workload("rows64", 1, 0, 8, 4, 128, "bf16", 32, (400,), 20, 0.2, 2, "recency",
                       budget_tokens=100.0, seed=35),
        synth.Workload("w128", 1, 0, 2, 2, 64, "bf16", 128, (900,), 20, 0.2, 2, "gauss",
                       budget_tokens=300.0, seed=36),
        # packed sequences of very different lengths, one shorter than a tile, one a single tile plus one key
        synth.Workload("packed_tc", 2, 0, 8, 2, 128, "bf16", 32, (100, 129, 1500, 128), 16, (0.05, 0.3), 2,
                       "recency", budget_frac=0.5, seed=37),
    ]
    for wl in cases:
        stats = run_and_check(wl)
        assert stats["units"] == (wl.n_layers - wl.n_shallow) * wl.batch * wl.n_kv_heads


def test_host_fed_pass_equals_resident_pass():
    # the streamed call (pinned host buffers in, pinned host buffers out, CodeBook layers in groups) must
    # return exactly what the resident call leaves on the device
    wl = synth.Workload("hostfed", 5, 3, 8, 2, 128, "bf16", 32, (600,), 20, (0.05, 0.3), 2, "recency",
                        budget_tokens=200.0, seed=41)
    host = generate(wl)
    layers = list(range(wl.n_layers))
    K, V = stack_layers(wl, host, layers, "K"), stack_layers(wl, host, layers, "V")
    Q = stack_layers(wl, host, layers[wl.n_shallow:], "Q")
    p = _pass(wl)
    p.run(K, V, Q)
    p2 = _pass(wl, layers_per_codebook_call=2)
    out = p2.host_outputs()
    hK, hV, hQ = K.cpu().pin_memory(), V.cpu().pin_memory(), Q.cpu().pin_memory()
    for _ in range(2):   # the second call reuses the staging buffers
        p2.run_from_host(hK, hV, hQ, out)
        torch.cuda.synchronize()
        for g in ("K", "V"):
            n = p.cb[g]["n_entries"].cpu()
            assert torch.equal(out[f"{g}.n_entries"], n)
            assert torch.equal(out[f"{g}.ref"], p.cb[g]["ref"].cpu())
            assert torch.equal(out[f"{g}.mag"], p.cb[g]["mag"].cpu())
            C = p.cb[g]["C"].cpu()
            for li in range(wl.n_shallow):
                for j in range(wl.n_kv_heads):
                    m = int(n[li, 0, j])
                    assert torch.equal(out[f"{g}.C"][li, 0, j, :m], C[li, 0, j, :m])
        assert torch.equal(out["keep_cnt"], p.keep_cnt.cpu())
        cnt = p.keep_cnt.cpu()
        for li in range(wl.n_layers - wl.n_shallow):
            for j in range(wl.n_kv_heads):
                m = int(cnt[li, 0, j])
                assert torch.equal(out["keep_idx"][li, j, :m], p.keep_idx.cpu()[li, j, :m])
                assert torch.equal(out["K_kept"][li, 0, j, :m], p.K_kept.cpu()[li, 0, j, :m])
                assert torch.equal(out["V_kept"][li, 0, j, :m], p.V_kept.cpu()[li, 0, j, :m])


def test_three_streams_give_what_one_stream_gives():
    # run() puts the K CodeBooks, the V CodeBooks and the eviction on three streams (two CodeBook workspaces);
    # every output must equal that of the three calls one after the other on one stream
    wl = synth.Workload("streams", 6, 3, 8, 2, 128, "bf16", 32, (700, 1300, 420), 30, (0.05, 0.3), 2, "recency",
                        budget_frac=0.3, seed=43)
    host = generate(wl)
    layers = list(range(wl.n_layers))
    K, V = stack_layers(wl, host, layers, "K"), stack_layers(wl, host, layers, "V")
    Q = stack_layers(wl, host, layers[wl.n_shallow:], "Q")
    serial = _pass(wl)
    serial.side_by_side = False
    serial.run(K, V, Q)
    side = _pass(wl)
    assert side.side_by_side
    for _ in range(2):   # the second run reuses the side streams and the second workspace
        side.run(K, V, Q)
        st = side.device_status()
        assert st["evict"][0] == 0 and st["codebook"][0] == 0 and st["codebook_v"][0] == 0
        for g in ("K", "V"):
            n = serial.cb[g]["n_entries"].cpu()
            assert torch.equal(side.cb[g]["n_entries"].cpu(), n)
            assert torch.equal(side.cb[g]["ref"], serial.cb[g]["ref"])
            assert torch.equal(side.cb[g]["mag"], serial.cb[g]["mag"])
            cu = synth.cu_seqlens(wl)
            for li in range(wl.n_shallow):
                for s_ in range(len(wl.seq_lens)):
                    for j in range(wl.n_kv_heads):
                        m = int(n[li, s_, j])
                        a, b = int(cu[s_]), int(cu[s_]) + m
                        assert torch.equal(side.cb[g]["centre_idx"][li, j, a:b], serial.cb[g]["centre_idx"][li, j, a:b])
                        assert torch.equal(side.cb[g]["C"][li, a:b, j], serial.cb[g]["C"][li, a:b, j])
        assert torch.equal(side.keep_cnt, serial.keep_cnt)
        cnt = serial.keep_cnt.cpu()
        for li in range(wl.n_layers - wl.n_shallow):
            for s_ in range(len(wl.seq_lens)):
                for j in range(wl.n_kv_heads):
                    m = int(cnt[li, s_, j])
                    a, b = int(cu[s_]), int(cu[s_]) + m
                    assert torch.equal(side.keep_idx[li, j, a:b], serial.keep_idx[li, j, a:b])
                    assert torch.equal(side.K_kept[li, a:b, j], serial.K_kept[li, a:b, j])
                    assert torch.equal(side.V_kept[li, a:b, j], serial.V_kept[li, a:b, j])


def test_a_pass_replayed_from_a_cuda_graph_gives_the_same_outputs():
    # run() recorded once (three streams, memsets and all kernels) and replayed on new contents of the same input tensors
    wl = synth.Workload("graph", 4, 2, 8, 2, 128, "bf16", 32, (900,), 30, (0.05, 0.3), 2, "recency",
                        budget_frac=0.3, seed=44)
    other = wl.replace(seed=45)
    layers = list(range(wl.n_layers))
    def tensors(w):
        host = generate(w)
        return (stack_layers(w, host, layers, "K"), stack_layers(w, host, layers, "V"),
                stack_layers(w, host, layers[w.n_shallow:], "Q"))
    K, V, Q = tensors(wl)
    K2, V2, Q2 = tensors(other)
    direct = _pass(wl)
    direct.run(K2, V2, Q2)
    p = _pass(wl)
    graph = p.capture(K, V, Q)
    K.copy_(K2); V.copy_(V2); Q.copy_(Q2)
    for _ in range(2):
        graph.replay()
        st = p.device_status()
        assert st["evict"][0] == 0 and st["codebook"][0] == 0 and st["codebook_v"][0] == 0
        for g in ("K", "V"):
            n = direct.cb[g]["n_entries"].cpu()
            assert torch.equal(p.cb[g]["n_entries"].cpu(), n)
            assert torch.equal(p.cb[g]["ref"], direct.cb[g]["ref"]) and torch.equal(p.cb[g]["mag"], direct.cb[g]["mag"])
            for li in range(wl.n_shallow):
                for j in range(wl.n_kv_heads):
                    m = int(n[li, 0, j])
                    assert torch.equal(p.cb[g]["C"][li, 0, j, :m], direct.cb[g]["C"][li, 0, j, :m])
        assert torch.equal(p.keep_cnt, direct.keep_cnt)
        cnt = direct.keep_cnt.cpu()
        for li in range(wl.n_layers - wl.n_shallow):
            for j in range(wl.n_kv_heads):
                m = int(cnt[li, 0, j])
                assert torch.equal(p.keep_idx[li, j, :m], direct.keep_idx[li, j, :m])
                assert torch.equal(p.K_kept[li, 0, j, :m], direct.K_kept[li, 0, j, :m])


def test_side_stream_of_the_composition_as_written_changes_nothing():
    # the literal and the repeat pass build the V CodeBooks on a side stream while the K CodeBooks are built on the
    # caller's: same outputs as one Gamma after the other
    from paper_2507_06517_b200.pipeline import SpindleKVLiteralPass, SpindleKVRepeatPass
    wl = synth.Workload("lits", 3, -1, 8, 2, 128, "bf16", 32, (900, 900), 30, (0.05, 0.3), 2, "recency",
                        budget_frac=0.3, seed=47)
    host = generate(wl)
    layers = list(range(wl.n_layers))
    K, V, Q = (stack_layers(wl, host, layers, x) for x in ("K", "V", "Q"))
    for cls in (SpindleKVLiteralPass, SpindleKVRepeatPass):
        a = cls(make_config(wl), wl.seq_lens, torch_dtype(wl))
        a.run(K, V, Q)                                   # K on the caller's stream, V on the side stream
        st = a.device_status()
        assert st["codebook"][0] == 0 and st["codebook_v"][0] == 0
        b = cls(make_config(wl), wl.seq_lens, torch_dtype(wl))
        b.run(K, V, Q, which=("K",))
        b.run(K, V, Q, which=("V",))
        torch.cuda.synchronize()
        for g in ("K", "V"):
            n = b.cb[g]["n_entries"].cpu()
            assert torch.equal(a.cb[g]["n_entries"].cpu(), n)
            assert torch.equal(a.cb[g]["ref"], b.cb[g]["ref"]) and torch.equal(a.cb[g]["mag"], b.cb[g]["mag"])
            for li in range(wl.n_layers):
                for s_ in range(len(wl.seq_lens)):
                    for j in range(wl.n_kv_heads):
                        m = int(n[li, s_, j])
                        assert torch.equal(a.cb[g]["C"][li, s_, j, :m], b.cb[g]["C"][li, s_, j, :m])


def test_composition_as_written_evict_then_codebooks_of_the_kept_tokens():
    # every layer evicts under the pyramid over all layers, then builds K and V CodeBooks of what it kept
    # (different counts per layer, passed to the CodeBook call as per-layer lengths)
    from paper_2507_06517_b200.pipeline import SpindleKVLiteralPass
    wl = synth.Workload("literal", 3, -1, 8, 2, 128, "bf16", 32, (700,), 12, (0.03, 0.3), 2, "recency",
                        budget_tokens=260.0, seed=51)
    layers = list(range(wl.n_layers))
    host = {lam: synth.layer_arrays(wl, lam, need_q=True) for lam in layers}
    K, V, Q = (stack_layers(wl, host, layers, x) for x in ("K", "V", "Q"))
    p = SpindleKVLiteralPass(make_config(wl), wl.seq_lens, torch_dtype(wl), keep_adjacency=True)
    _, _, k_plan = O.plan_layers(wl.n_layers, -1, wl.seq_lens, wl.window, wl.beta, budget_tokens=wl.budget_tokens)
    assert np.array_equal(k_plan, p.k_ctx_host) and len(set(k_plan[:, 0])) == wl.n_layers
    H, l, w = wl.n_kv_heads, wl.max_len, wl.window
    units = 0
    for g, idx, theta in (("K", 0, wl.theta_k), ("V", 1, wl.theta_v)):
        p.run(K, V, Q, which=(g,))
        st = p.device_status()
        assert st["evict"][0] == 0 and st["codebook"][0] == 0 and st["codebook"][1][1] == 0
        keep = p.ev.keep_idx.cpu().numpy()
        cnt = p.ev.keep_cnt.cpu().numpy()
        scores = p.ev.scores.cpu().numpy()
        o = {k: (v.float() if k == "C" else v).cpu().numpy() for k, v in p.cb[g].items()}
        adj = p.adj.cpu().numpy()
        for lam in layers:
            k_ctx = int(k_plan[lam, 0])
            Ks = np.stack([host[lam][0][0, j] for j in range(H)])
            check_evict_unit(wl, host[lam][2][0], Ks, k_ctx, scores[lam], keep[lam], cnt[lam, 0])
            n = k_ctx + w
            for j in range(H):
                # the checker builds its CodeBook from the rows this layer and head actually kept
                gamma = host[lam][idx][0, j][keep[lam, j, :n]]
                check_codebook_unit(gamma, theta, adj[lam * H + j], o["mag"][lam, j, :n],
                                    o["ref"][lam, j, :n], o["centre_idx"][lam, j, :n], int(o["n_entries"][lam, 0, j]),
                                    o["C"][lam, 0, j], value_tol(wl))
                units += 1
    assert units == 2 * wl.n_layers * H
    nk, nv = p.entry_counts()
    for lam in layers:   # Eq. (15)
        r1, r2 = O.reserve_ratio_layer(l, int(k_plan[lam, 0]) + w, nk[lam, 0], nv[lam, 0])
        assert 0 < r1 <= 1 and 0 < r2 <= 1


def test_gqa_repeat_variant():
    # every query head selects on its own; the CodeBooks of a KV head are built from all its query heads' tokens
    from paper_2507_06517_b200.pipeline import SpindleKVRepeatPass
    wl = synth.Workload("repeat", 2, -1, 8, 2, 128, "bf16", 32, (640,), 12, (0.03, 0.3), 2, "recency",
                        budget_tokens=150.0, seed=71)
    layers = list(range(wl.n_layers))
    host = {lam: synth.layer_arrays(wl, lam, need_q=True) for lam in layers}
    K, V, Q = (stack_layers(wl, host, layers, x) for x in ("K", "V", "Q"))
    p = SpindleKVRepeatPass(make_config(wl), wl.seq_lens, torch_dtype(wl), keep_adjacency=True)
    _, _, k_plan = O.plan_layers(wl.n_layers, -1, wl.seq_lens, wl.window, wl.beta, budget_tokens=wl.budget_tokens)
    H, h_n, l, w = wl.n_kv_heads, wl.group, wl.max_len, wl.window
    one = wl.replace(n_q_heads=H)   # a group of one query head per KV head, as each eviction call sees it
    for g, idx, theta in (("K", 0, wl.theta_k), ("V", 1, wl.theta_v)):
        p.run(K, V, Q, which=(g,))
        st = p.device_status()
        assert st["evict"][0] == 0 and st["codebook"][0] == 0 and st["codebook"][1][1] == 0
        keep, cnt, scores = p.keep_idx.cpu().numpy(), p.keep_cnt.cpu().numpy(), p.scores.cpu().numpy()   # per query head
        union, ucnt = p.union_idx.cpu().numpy(), p.union_cnt.cpu().numpy()
        o = {k: (v.float() if k == "C" else v).cpu().numpy() for k, v in p.cb[g].items()}
        adj = p.adj.cpu().numpy()
        for lam in layers:
            k_ctx = int(k_plan[lam, 0])
            n = k_ctx + w
            Ks = np.stack([host[lam][0][0, j] for j in range(H)])
            for gq in range(h_n):
                # the query heads at position gq of every group, each against its own KV head: a group of one
                sel = np.arange(gq, wl.n_q_heads, h_n)
                check_evict_unit(one, host[lam][2][0][sel], Ks, k_ctx, scores[lam][sel], keep[lam][sel], cnt[lam, 0][sel])
            for j in range(H):
                assert ucnt[lam, 0, j] == h_n * n
                want_union = np.concatenate([keep[lam, h_n * j + gq, :n] for gq in range(h_n)])
                assert np.array_equal(union[lam, j, : h_n * n], want_union)
                gamma = host[lam][idx][0, j][want_union]
                check_codebook_unit(gamma, theta, adj[lam * H + j], o["mag"][lam, j, : h_n * n], o["ref"][lam, j, : h_n * n],
                                    o["centre_idx"][lam, j, : h_n * n], int(o["n_entries"][lam, 0, j]), o["C"][lam, 0, j],
                                    value_tol(wl))
                # copies of a token share an entry
                ref = o["ref"][lam, j, : h_n * n]
                for tok in np.unique(want_union):
                    assert len(set(ref[want_union == tok])) == 1


def test_per_query_head_eviction_on_every_window_shape():
    # Section 3.3's alternative to the group mean, one call: every query head gets its own score row (Eq. (2)) and its
    # own kept set; windows of 16 (two heads per 32-column chunk), 32, 64 (two chunks per head), 256 query rows per
    # KV head, and the fp32 CUDA-core kernels
    from paper_2507_06517_b200 import binding as B
    cases = [
        synth.Workload("pq_w32", 2, 0, 8, 2, 128, "bf16", 32, (900,), 20, (0.05, 0.3), 2, "recency", budget_tokens=200.0, seed=111),
        synth.Workload("pq_w16", 1, 0, 16, 4, 64, "bf16", 16, (640,), 20, 0.2, 2, "recency", budget_tokens=100.0, seed=112),
        synth.Workload("pq_w64", 1, 0, 8, 2, 128, "bf16", 64, (1100,), 30, (0.05, 0.3), 4, "recency", budget_tokens=300.0, seed=113),
        synth.Workload("pq_qb2", 1, 0, 16, 2, 64, "bf16", 32, (700,), 30, (0.05, 0.3), 4, "recency", budget_tokens=200.0, seed=114),
        synth.Workload("pq_f32", 1, 0, 4, 2, 64, "f32", 32, (333,), 8, 0.1, 2, "gauss", budget_tokens=80.0, seed=115),
    ]
    for wl in cases:
        host = generate(wl)
        layers = list(range(wl.n_layers))
        K, Q = stack_layers(wl, host, layers, "K"), stack_layers(wl, host, layers, "Q")
        cfg = make_config(wl, per_query_head=1)
        L, Hq, H, N, w, h_n = wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.max_len, wl.window, wl.group
        batch = B.Batch(L, 1, N, N)
        _, _, k_plan = B.spindlekv_plan_layers(cfg, wl.seq_lens)
        k_dev = torch.from_numpy(np.ascontiguousarray(k_plan)).cuda()
        keep = torch.full((L, Hq, N), -1, dtype=torch.int32, device="cuda")
        cnt = torch.zeros((L, 1, Hq), dtype=torch.int32, device="cuda")
        scores = torch.zeros((L, Hq, N), dtype=torch.float32, device="cuda")
        ws = torch.empty(B.spindlekv_workspace_bytes(cfg, batch, B.WS_EVICT), dtype=torch.uint8, device="cuda")
        B.spindlekv_evict_deep(cfg, batch, B.desc_bhnd(K), B.desc_bhnd(Q), k_dev, keep, cnt, scores, ws)
        torch.cuda.synchronize()
        assert B.spindlekv_poll_status(ws)[0] == 0
        keep, cnt, scores = keep.cpu().numpy(), cnt.cpu().numpy(), scores.cpu().numpy()
        one = wl.replace(n_q_heads=1, n_kv_heads=1)
        for lam in layers:
            for i in range(Hq):
                check_evict_unit(one, host[lam][2][0][i:i + 1], host[lam][0][0][i // h_n:i // h_n + 1], int(k_plan[lam, 0]),
                                 scores[lam, i:i + 1], keep[lam, i:i + 1], cnt[lam, 0, i:i + 1])


def test_decode_time_merge_into_existing_codebooks():
    # CodeBooks of the first tokens of a sequence, then the rest of the sequence arrives as new tokens: some
    # find an entry, the others get entries of their own, appended
    from paper_2507_06517_b200 import binding as B
    from paper_2507_06517_b200.pipeline import SpindleKVDecodeMerge
    for dtype, d, l0, t_new, tol in (("bf16", 128, 512, 200, 1e-2), ("f32", 64, 300, 90, 1e-5)):
        wl = synth.Workload("merge", 2, 2, 4, 2, d, dtype, 8, (l0 + t_new,), 24, (0.03, 0.3), 2, "gauss",
                            budget_tokens=float(l0 + t_new), seed=81)
        host = generate(wl)
        full = stack_layers(wl, host, [0, 1], "K")                      # [2, 1, H, l0 + t_new, d]
        old, new = full[:, :, :, :l0].contiguous(), full[:, :, :, l0:].contiguous()
        H, theta, c_rows = wl.n_kv_heads, wl.theta_k, l0 + t_new
        base = synth.Workload("base", 2, 2, 4, 2, d, dtype, 8, (l0,), 24, 0.1, 2, "gauss", budget_tokens=float(l0))
        p = _pass(base)
        p.codebook(old, "K")
        C = torch.zeros((2, 1, H, c_rows, d), dtype=old.dtype, device="cuda")
        C[:, :, :, :l0] = p.cb["K"]["C"]
        n_entries = p.cb["K"]["n_entries"].clone()
        C_before, n_before = C.float().cpu().numpy(), n_entries.cpu().numpy()
        m = SpindleKVDecodeMerge(make_config(base), 2, 1, t_new, c_rows, old.dtype, keep_adjacency=True)
        m.run(new, C, n_entries, theta)
        torch.cuda.synchronize()
        assert B.spindlekv_poll_status(m.ws_codebook)[0] == 0
        ref, mag, left_idx, left_cnt = (x.cpu().numpy() for x in (m.ref_new, m.mag_new, m.left_idx, m.left_cnt))
        C_after, n_after, adj = C.float().cpu().numpy(), n_entries.cpu().numpy(), m.adj.cpu().numpy()
        sub = {k: v.cpu().numpy() for k, v in m.left.items()}
        new_h = new.float().cpu().numpy()
        n_near = n_matched = n_unmatched = 0
        for li in range(2):
            for j in range(H):
                n0 = int(n_before[li, 0, j])
                gam = new_h[li, 0, j]
                want_ref, S = O.match_entries(C_before[li, 0, j, :n0], gam, theta)
                got = ref[li, j]
                np.testing.assert_allclose(mag[li, j], O.magnitudes(gam), rtol=2e-6)
                matched = np.array([got[t] if 0 <= got[t] < n0 else -1 for t in range(t_new)])
                for t in range(t_new):
                    top = S[t].max()
                    if matched[t] != want_ref[t]:
                        n_near += 1   # only on the threshold, or between entries that are equally similar
                        if matched[t] < 0 or want_ref[t] < 0:
                            assert abs(top - theta) < REL_MARGIN * theta
                        else:
                            assert S[t, matched[t]] > top - REL_MARGIN * abs(top)
                left = np.flatnonzero(matched < 0)
                n_matched += t_new - left.size
                n_unmatched += left.size
                assert left_cnt[li, 0, j] == left.size and np.array_equal(left_idx[li, j, : left.size], left)
                # the unmatched tokens' own CodeBook, against the checker on the same rows
                unit = li * H + j
                n_add = int(sub["n_entries"][li, 0, j])
                if left.size:
                    check_codebook_unit(gam[left], theta, adj[unit], sub["mag"][li, j, : left.size], sub["ref"][li, j, : left.size],
                                        sub["centre_idx"][li, j, : left.size], n_add, None, tol)
                    assert np.array_equal(got[left], n0 + sub["ref"][li, j, : left.size])
                    rows = gam[left][sub["centre_idx"][li, j, :n_add]].astype(np.float64)
                    np.testing.assert_allclose(C_after[li, 0, j, n0:n0 + n_add], rows / np.linalg.norm(rows, axis=1, keepdims=True),
                                               rtol=tol, atol=tol)
                assert n_after[li, 0, j] == n0 + n_add
                assert np.array_equal(C_after[li, 0, j, :n0], C_before[li, 0, j, :n0])       # old entries untouched
                # every new token ends up within the threshold of its entry (Eq. (14))
                ent = C_after[li, 0, j][got].astype(np.float64)
                cos = (ent * gam).sum(1) / (np.linalg.norm(ent, axis=1) * np.linalg.norm(gam, axis=1))
                assert np.all(cos > theta - 2 * tol)
        assert (ref >= 0).all() and n_matched > 0 and n_unmatched > 0   # both branches were exercised


def test_reconstruction_from_the_codebook():
    # Eq. (14): C[r] (x) m, against the checker's reconstruction from the same CodeBook rows; and the
    # reconstructed rows keep each token's magnitude and a cosine above the threshold to the original
    from paper_2507_06517_b200 import binding as B
    for wl in (synth.Workload("rec32", 2, 2, 2, 2, 64, "f32", 8, (300, 300), 10, 0.1, 2, "gauss", budget_tokens=300.0, seed=61),
               synth.Workload("rec16", 1, 1, 4, 2, 128, "bf16", 8, (333, 700, 128), 16, (0.03, 0.2), 2, "gauss",
                              budget_frac=1.0, seed=62)):
        host = generate(wl)
        p = _pass(wl)
        K = stack_layers(wl, host, list(range(wl.n_shallow)), "K")
        p.codebook(K, "K")
        o = p.cb["K"]
        out = torch.zeros_like(K)
        B.spindlekv_reconstruct(p.cb_batch, wl.n_kv_heads, wl.head_dim, p._desc(o["C"]), o["ref"], o["mag"], p._desc(out))
        torch.cuda.synchronize()
        got, Cn, ref, mag = out.float().cpu().numpy(), o["C"].float().cpu().numpy(), o["ref"].cpu().numpy(), o["mag"].cpu().numpy()
        tol = value_tol(wl)
        for li in range(wl.n_shallow):
            for s, l in enumerate(wl.seq_lens):
                tb = tok_base(wl, s)
                for j in range(wl.n_kv_heads):
                    want = O.reconstruct(unit_rows(wl, Cn[li], s, j), ref[li, j, tb:tb + l], mag[li, j, tb:tb + l])
                    rows = unit_rows(wl, got[li], s, j)[:l]
                    np.testing.assert_allclose(rows, want, rtol=tol, atol=tol * np.abs(want).max())
                    orig = unit_rows(wl, host[li][0], s, j).astype(np.float64)
                    cos = (rows * orig).sum(1) / (np.linalg.norm(rows, axis=1) * np.linalg.norm(orig, axis=1))
                    assert np.all(cos > wl.theta_k - 2 * tol)
                    np.testing.assert_allclose(np.linalg.norm(rows, axis=1), mag[li, j, tb:tb + l], rtol=2 * tol)


def test_plain_window_sum_extension():
    wl = synth.Workload("rawsum", 1, 0, 4, 2, 64, "f32", 32, (333,), 8, 0.1, 2, "gauss", budget_tokens=80.0, seed=14)
    run_and_check(wl, {"score_norm": 1})


def test_keep_everything_and_minimum_budget():
    wl = synth.Workload("all", 1, 0, 4, 2, 64, "f32", 32, (160,), 8, 0.1, 2, "gauss", budget_tokens=160.0, seed=15)
    run_and_check(wl)  # r_c = 1: every context token kept
    wl = wl.replace(budget_tokens=32 + 0.051 * 128)  # just above beta: k = floor(0.051 * 128) = 6
    run_and_check(wl)


def _single_layer_codebook(gamma_np, theta, dtype="f32", keep_adjacency=True, poison=False):
    """Runs the CodeBook path on one hand-made ``[l, d]`` array; returns outputs as numpy.  ``poison`` fills the
    workspace with a byte pattern first (nothing in it may be taken for initialised)."""
    l, d = gamma_np.shape
    wl = synth.Workload("hand", 1, 1, 1, 1, d, dtype, 1, (l,), 1, 0.1, 0, "gauss", budget_tokens=float(l),
                        theta_k=theta, theta_v=theta)
    p = _pass(wl, keep_adjacency=keep_adjacency)
    if poison:
        p.ws_codebook.fill_(0xA5)
    G = torch.from_numpy(gamma_np.astype(np.float32)).to(torch_dtype(wl)).cuda().reshape(1, 1, 1, l, d)
    p.codebook(G, "K")
    assert p.device_status()["codebook"][0] == 0
    o = p.cb["K"]
    return (p.adj.cpu().numpy()[0] if keep_adjacency else None, o["mag"].cpu().numpy()[0, 0], o["ref"].cpu().numpy()[0, 0],
            o["centre_idx"].cpu().numpy()[0, 0], int(o["n_entries"].cpu().numpy()[0, 0, 0]),
            o["C"].float().cpu().numpy()[0, 0, 0])


def test_degenerate_thresholds_duplicates_and_zero_rows():
    rng = np.random.default_rng(21)
    g = rng.standard_normal((150, 64)).astype(np.float32)
    adj, mag, ref, cen, n, C = _single_layer_codebook(g, 1.5)  # nobody similar: identity CodeBook
    assert n == 150 and list(cen[:150]) == list(range(150)) and list(ref[:150]) == list(range(150))
    adj, mag, ref, cen, n, C = _single_layer_codebook(g, -1.5)  # everybody similar: one entry, centre 0
    assert n == 1 and cen[0] == 0 and np.all(ref[:150] == 0)
    base = rng.standard_normal((50, 64)).astype(np.float32)
    g = np.concatenate([base, 2.0 * base, base])  # exact copies (cosine 1) collapse
    g[7] = 0.0  # a zero vector keeps an entry of its own
    out = _single_layer_codebook(g, 0.999)
    check_codebook_unit(g, 0.999, *out, 1e-5)
    assert out[4] == 50 + 1 + 0  # 49 shared entries + the zero row + row 57/107 pair still shares one


def test_degenerate_cases_on_the_tensor_core_path():
    rng = np.random.default_rng(22)
    from paper_2507_06517_b200.synth import round_to_dtype
    for d, n in ((128, 700), (64, 300)):
        g = round_to_dtype(rng.standard_normal((n, d)).astype(np.float32), "bf16")
        adj, mag, ref, cen, cnt, C = _single_layer_codebook(g, 1.5, "bf16")
        assert cnt == n and list(cen[:n]) == list(range(n)) and list(ref[:n]) == list(range(n))
        g[5] = 0.0
        g[n - 1] = 0.0
        out = _single_layer_codebook(g, -1.5, "bf16")  # zero rows have similarity 0 > theta with everybody
        assert out[4] == 1 and np.all(out[2][:n] == 0)
        base = round_to_dtype(rng.standard_normal((n // 3, d)).astype(np.float32), "bf16")
        g = np.concatenate([base, 2.0 * base, base, base[: n - 3 * (n // 3)]])
        g[7] = 0.0
        out = _single_layer_codebook(g, 0.999, "bf16")
        check_codebook_unit(g, 0.999, *out, 1e-2)


def test_tensor_core_similarity_at_awkward_lengths():
    # lengths around the 128-row blocks and 256-row spans of the CTA pairs (odd numbers of blocks, a lone block,
    # two tokens), both head sizes; clustered rows so that the graphs are not empty
    rng = np.random.default_rng(23)
    from paper_2507_06517_b200.synth import round_to_dtype
    for d in (128, 64):
        for n in (2, 31, 128, 129, 255, 256, 257, 383, 385, 641, 1100):
            cents = rng.standard_normal((max(2, n // 12), d)).astype(np.float32)
            g = cents[rng.integers(0, cents.shape[0], size=n)] + 0.12 * rng.standard_normal((n, d)).astype(np.float32)
            g = round_to_dtype(g, "bf16")
            out = _single_layer_codebook(g, 0.95, "bf16")
            check_codebook_unit(g, 0.95, *out, 1e-2)


def test_adjacency_in_a_poisoned_workspace_with_dense_rows():
    # When the adjacency lives in the caller's workspace, chunks of it without a set bit are never written and
    # must never be read: the workspace is filled with a byte pattern first.  Groups of 40 to 70 exactly parallel
    # rows (power-of-two multiples: cosine 1) give rows with more than 32 neighbours, which are read as whole bit
    # rows; everything else is far from the threshold, so the result is the checker's without any margin.
    rng = np.random.default_rng(24)
    from paper_2507_06517_b200.synth import round_to_dtype
    for d, n in ((128, 1500), (64, 900)):
        dirs = round_to_dtype(rng.standard_normal((40, d)).astype(np.float32), "bf16")
        sizes = list(rng.integers(40, 71, size=6)) + [1] * 34
        rows = []
        for c, sz in enumerate(sizes):
            rows += [dirs[c] * (2.0 ** int(e)) for e in rng.integers(-2, 3, size=sz)]
        while len(rows) < n:
            rows.append(round_to_dtype(rng.standard_normal(d).astype(np.float32), "bf16"))
        g = np.stack(rows)[rng.permutation(len(rows))][:n]
        out = _single_layer_codebook(g, 0.9, "bf16", keep_adjacency=False, poison=True)
        check_codebook_unit(g, 0.9, *out, 1e-2)
        ref = _single_layer_codebook(g, 0.9, "bf16")
        assert np.array_equal(out[2], ref[2]) and np.array_equal(out[3], ref[3]) and out[4] == ref[4]


def test_all_scores_tie_goes_to_lowest_positions():
    # zero queries: plain window sums tie everywhere -> the first k context tokens; with the division
    # by (l - a) scores rise with position -> the last k
    wl = synth.Workload("tie", 1, 0, 2, 1, 64, "f32", 16, (200,), 4, 0.1, 0, "gauss", budget_tokens=56.0, seed=16)
    host = generate(wl)
    l_c, k = 200 - 16, 40
    for norm, want in ((1, list(range(k))), (0, list(range(l_c - k, l_c)))):
        p = _pass(wl, cfg={"score_norm": norm})
        K = stack_layers(wl, host, [0], "K")
        Q = torch.zeros((1, 1, 2, 16, 64), dtype=torch.float32, device="cuda")
        p.evict(K, K, Q)
        keep = p.keep_idx.cpu().numpy()[0, 0]
        assert list(keep[:k]) == want and list(keep[k:k + 16]) == list(range(l_c, 200))
