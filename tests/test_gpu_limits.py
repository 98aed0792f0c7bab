"""The paths behind the library's limits, reached by tightening the limits (never by faulting or hanging
a GPU): units whose candidate pairs do not fit the record pool are computed as a bit matrix and must give
the very same CodeBooks; a bounded wait that runs out must come back with TIMEOUT in the status word and
leave the device usable."""
import numpy as np
import pytest
import torch

from paper_2507_06517_b200 import synth

from gpu_util import check_codebook_unit, generate, make_config, stack_layers, torch_dtype, value_tol

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _restore_limits():
    from paper_2507_06517_b200 import binding as B
    yield
    for k in range(4):
        B.spindlekv_set_tuning(k, -1)


def _codebooks(wl, which="K", poison=False):
    from paper_2507_06517_b200.pipeline import SpindleKVPass
    host = generate(wl)
    p = SpindleKVPass(make_config(wl), wl.seq_lens, torch_dtype(wl), keep_adjacency=True)
    if poison:
        p.ws_codebook.fill_(0xA5)
    G = stack_layers(wl, host, list(range(wl.n_shallow)), which)
    p.codebook(G, which)
    status, detail = p.device_status()["codebook"]
    assert status == 0 and detail[1] == 0
    o = p.cb[which]
    out = {k: (v.float() if k == "C" else v).cpu().numpy() for k, v in o.items()}
    out["adj"] = p.adj.cpu().numpy()
    return host, out, detail[2]


def test_units_that_overflow_the_record_pool_fall_back_to_the_bit_matrix():
    from paper_2507_06517_b200 import binding as B
    wl = synth.Workload("paths", 2, 2, 8, 2, 128, "bf16", 32, (1100,), 150, (0.05, 0.3), 4, "recency",
                        budget_tokens=1100.0, seed=91)
    units = wl.n_shallow * wl.n_kv_heads
    host, ref_out, n_bits = _codebooks(wl, "V")
    assert n_bits == 0                                    # the default pool holds every unit of this sparse case
    for li in range(wl.n_shallow):
        for j in range(wl.n_kv_heads):
            check_codebook_unit(host[li][1][0, j], wl.theta_v, ref_out["adj"][li * wl.n_kv_heads + j], ref_out["mag"][li, j],
                                ref_out["ref"][li, j], ref_out["centre_idx"][li, j], int(ref_out["n_entries"][li, 0, j]),
                                ref_out["C"][li, 0, j], value_tol(wl))
    seen = []
    for cap in (2, 0):                                    # 2 records per tile: far below the pair count; 0: no records at all
        B.spindlekv_set_tuning(B.TUNE_RECORDS_PER_TILE, cap)
        _, out, n_bits = _codebooks(wl, "V", poison=True)
        seen.append(n_bits)
        for k in ("adj", "mag", "ref", "n_entries"):
            assert np.array_equal(out[k], ref_out[k]), k
        n = ref_out["n_entries"]
        for li in range(wl.n_shallow):
            for j in range(wl.n_kv_heads):
                m = int(n[li, 0, j])
                assert np.array_equal(out["centre_idx"][li, j, :m], ref_out["centre_idx"][li, j, :m])
                assert np.array_equal(out["C"][li, 0, j, :m], ref_out["C"][li, 0, j, :m])
    assert seen == [units, units]


def test_some_units_in_the_pool_and_some_through_the_bit_matrix_in_one_call():
    # layer 0 is almost free of similar pairs (noise far above the threshold), layer 1 is the clustered case: with a
    # small pool only the units of layer 1 overflow
    from paper_2507_06517_b200 import binding as B
    from paper_2507_06517_b200.pipeline import SpindleKVPass
    sparse = synth.Workload("s", 1, 1, 4, 2, 128, "bf16", 32, (900,), 30, 0.5, 2, "gauss", budget_tokens=900.0, seed=92)
    dense = synth.Workload("d", 1, 1, 4, 2, 128, "bf16", 32, (900,), 150, 0.1, 2, "gauss", budget_tokens=900.0, seed=93)
    G = torch.cat([stack_layers(sparse, generate(sparse), [0], "K"), stack_layers(dense, generate(dense), [0], "K")])
    two = sparse.replace(n_layers=2, n_shallow=2)
    outs = []
    for cap in (-1, 8):
        B.spindlekv_set_tuning(B.TUNE_RECORDS_PER_TILE, cap)
        p = SpindleKVPass(make_config(two), two.seq_lens, torch_dtype(two), keep_adjacency=True)
        p.codebook(G, "K")
        status, detail = p.device_status()["codebook"]
        assert status == 0 and detail[2] == (0 if cap < 0 else 2)
        outs.append([p.cb["K"][k].clone() for k in ("ref", "n_entries", "mag")] + [p.adj.clone()])
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    Gh = G.float().cpu().numpy()
    adj = outs[0][3].cpu().numpy()
    o = {k: (v.float() if k == "C" else v).cpu().numpy() for k, v in p.cb["K"].items()}
    for li in range(2):
        for j in range(2):
            check_codebook_unit(Gh[li, 0, j], two.theta_k, adj[li * 2 + j], o["mag"][li, j], o["ref"][li, j], o["centre_idx"][li, j],
                                int(o["n_entries"][li, 0, j]), o["C"][li, 0, j], 1e-2)


def test_more_overflowed_units_than_the_bit_matrix_pass_has_slots():
    # 48 units of two different lengths all overflow a tiny pool: every pair of blocks of the bit-matrix pass then
    # works through several units one after the other (ring stages and barrier phases carry on from unit to unit)
    from paper_2507_06517_b200 import binding as B
    from paper_2507_06517_b200.pipeline import SpindleKVPass
    wl = synth.Workload("many", 3, 3, 16, 8, 128, "bf16", 32, (700, 390), 100, (0.05, 0.3), 2, "recency",
                        budget_frac=1.0, seed=94)
    host = generate(wl)
    G = stack_layers(wl, host, [0, 1, 2], "V")
    units = wl.n_shallow * wl.batch * wl.n_kv_heads
    outs = []
    for cap in (-1, 2):
        B.spindlekv_set_tuning(B.TUNE_RECORDS_PER_TILE, cap)
        p = SpindleKVPass(make_config(wl), wl.seq_lens, torch_dtype(wl), keep_adjacency=True)
        p.ws_codebook.fill_(0x5A)
        p.codebook(G, "V")
        status, detail = p.device_status()["codebook"]
        assert status == 0 and detail[2] == (0 if cap < 0 else units)
        outs.append([p.cb["V"][k].clone() for k in ("ref", "n_entries", "mag")] + [p.adj.clone()])
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    # and the result is the checker's (one unit of each length)
    o = {k: (v.float() if k == "C" else v).cpu().numpy() for k, v in p.cb["V"].items()}
    adj = outs[1][3].cpu().numpy()
    cu = synth.cu_seqlens(wl)
    for li, s_, j in ((0, 0, 0), (2, 1, 7)):
        l = wl.seq_lens[s_]
        unit = (li * wl.batch + s_) * wl.n_kv_heads + j
        gamma = host[li][1][cu[s_]:cu[s_ + 1], j]
        check_codebook_unit(gamma, wl.theta_v, adj[unit], o["mag"][li, j, cu[s_]:cu[s_] + l], o["ref"][li, j, cu[s_]:cu[s_] + l],
                            o["centre_idx"][li, j, cu[s_]:cu[s_] + l], int(o["n_entries"][li, s_, j]), None, 1e-2)


def test_few_block_pairs_walk_every_unit_and_row_span():
    # The candidate-record kernel runs a fixed number of block pairs that share out the (unit, pair of row spans) items.
    # With 1, 2 or 3 pairs every pair walks many items of sequences of different lengths (odd and even numbers of
    # 256-row spans, a last span with one live block only) and must give what the full grid gives.
    from paper_2507_06517_b200 import binding as B
    wl = synth.Workload("walk", 4, 2, 8, 2, 128, "bf16", 32, (1100, 300, 1537, 700), 120, (0.05, 0.3), 4, "recency",
                        budget_frac=0.3, seed=95)
    _, ref_out, n_bits = _codebooks(wl, "K")     # the full grid (checked against the oracle by the parity tests)
    assert n_bits == 0
    for pairs in (1, 2, 3):
        B.spindlekv_set_tuning(B.TUNE_SIM_BLOCK_PAIRS, pairs)
        assert B.spindlekv_get_tuning(B.TUNE_SIM_BLOCK_PAIRS) == pairs
        _, out, n_bits = _codebooks(wl, "K", poison=True)
        assert n_bits == 0
        for k in ("mag", "ref", "n_entries"):
            assert np.array_equal(out[k], ref_out[k]), (pairs, k)
        cu = synth.cu_seqlens(wl)
        for li in range(wl.n_shallow):
            for s_ in range(len(wl.seq_lens)):
                for j in range(wl.n_kv_heads):
                    m = int(ref_out["n_entries"][li, s_, j])
                    assert np.array_equal(out["centre_idx"][li, j, cu[s_]:cu[s_] + m], ref_out["centre_idx"][li, j, cu[s_]:cu[s_] + m])
        for u in range(ref_out["adj"].shape[0]):
            lu = wl.seq_lens[(u // wl.n_kv_heads) % len(wl.seq_lens)]
            assert np.array_equal(out["adj"][u, :lu, :(lu + 31) // 32], ref_out["adj"][u, :lu, :(lu + 31) // 32]), (pairs, u)


def test_dense_graph_goes_through_the_bit_matrix_by_itself():
    # three big clusters: rows with hundreds of neighbours, whose lists do not fit the record path's budget
    wl = synth.Workload("dense", 1, 1, 2, 2, 128, "bf16", 8, (700,), 3, (0.02, 0.1), 2, "gauss",
                        budget_tokens=700.0, seed=17)
    host, out, n_bits = _codebooks(wl, "K")
    assert n_bits == wl.n_kv_heads
    for j in range(wl.n_kv_heads):
        check_codebook_unit(host[0][0][0, j], wl.theta_k, out["adj"][j], out["mag"][0, j], out["ref"][0, j],
                            out["centre_idx"][0, j], int(out["n_entries"][0, 0, j]), out["C"][0, 0, j], 1e-2)


def test_bounded_waits_run_out_and_report_timeout():
    from paper_2507_06517_b200 import binding as B
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    B.spindlekv_selftest_mbarrier_timeout(ws, 20000)      # about ten microseconds of SM clock
    torch.cuda.synchronize()
    status, detail = B.spindlekv_poll_status(ws)
    assert status == B.TIMEOUT and detail[1] == 0
    # the device is as usable as before: an ordinary call gives the ordinary result
    wl = synth.workload("C1")
    host, out, _ = _codebooks(wl, "K")
    for j in range(wl.n_kv_heads):
        check_codebook_unit(host[0][0][0, j], wl.theta_k, out["adj"][j], out["mag"][0, j], out["ref"][0, j],
                            out["centre_idx"][0, j], int(out["n_entries"][0, 0, j]), out["C"][0, 0, j], value_tol(wl))


def test_greedy_cover_that_is_cut_short_reports_it():
    # a chain 0-1-2-...: the exact cover needs several rounds; with the cap at one round the kernel must stop, say
    # TIMEOUT, count the tokens it left without a centre, and write nothing out of bounds
    from paper_2507_06517_b200 import binding as B
    from paper_2507_06517_b200.pipeline import SpindleKVPass
    n, d = 96, 64
    ang = 0.1 * np.arange(n)
    g = np.zeros((n, d), dtype=np.float32)
    g[:, 0], g[:, 1] = np.cos(ang), np.sin(ang)           # neighbours 0.1 rad apart: cos 0.995 > theta, two apart 0.980 < theta
    theta = 0.99
    wl = synth.Workload("chain", 1, 1, 1, 1, d, "f32", 1, (n,), 1, 0.1, 0, "gauss", budget_tokens=float(n),
                        theta_k=theta, theta_v=theta)
    G = torch.from_numpy(g).cuda().reshape(1, 1, 1, n, d)
    p = SpindleKVPass(make_config(wl), wl.seq_lens, torch.float32, keep_adjacency=True)
    guard = torch.full((3, 64), -7, dtype=torch.int32, device="cuda")
    B.spindlekv_set_tuning(B.TUNE_GREEDY_ROUND_CAP, 1)
    p.codebook(G, "K")
    status, detail = p.device_status()["codebook"]
    assert status == B.TIMEOUT and detail[1] > 0
    assert torch.all(guard == -7)
    B.spindlekv_set_tuning(B.TUNE_GREEDY_ROUND_CAP, -1)
    p.codebook(G, "K")                                     # the same buffers, no cap: the exact result
    status, detail = p.device_status()["codebook"]
    assert status == B.OK and detail[1] == 0 and detail[0] > 2
    o = p.cb["K"]
    check_codebook_unit(g, theta, p.adj.cpu().numpy()[0], o["mag"].cpu().numpy()[0, 0], o["ref"].cpu().numpy()[0, 0],
                        o["centre_idx"].cpu().numpy()[0, 0], int(o["n_entries"].cpu().numpy()[0, 0, 0]),
                        o["C"].float().cpu().numpy()[0, 0, 0], 1e-5)
