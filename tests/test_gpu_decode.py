"""Decode-time attention over the replaced cache (Eq. (14) inside Eq. (1), rotary embedding re-applied) against the
CPU checker, through the C ABI.  The checker is given the CodeBook rows, references and magnitudes the GPU pass
produced (rows as stored, i.e. rounded to the storage type), so what is compared is the attention arithmetic:
outputs within 1e-2 (bf16 rows) or 2e-5 (fp32 rows) of the largest output element."""
import numpy as np
import pytest
import torch

from oracle import spindlekv_oracle as O
from paper_2507_06517_b200 import synth

from gpu_util import generate, make_config, stack_layers, torch_dtype

pytestmark = pytest.mark.gpu


def _check(wl, out, q, pos_q, cbk, cbv, positions, base, tol):
    H, h_n = wl.n_kv_heads, wl.group
    Ck, Cv = cbk["C"].float().cpu().numpy(), cbv["C"].float().cpu().numpy()
    rk, mk, rv, mv = (x.cpu().numpy() for x in (cbk["ref"], cbk["mag"], cbv["ref"], cbv["mag"]))
    nk, nv = cbk["n_entries"].cpu().numpy(), cbv["n_entries"].cpu().numpy()
    got = out.cpu().numpy()
    qh = q.float().cpu().numpy()
    worst = 0.0
    for li in range(cbk["ref"].shape[0]):
        for s, l in enumerate(wl.seq_lens):
            tb = s * wl.max_len
            for j in range(H):
                n = l if positions is None else int(positions["len"][li, s])
                pos = None if positions is None else positions["pos"][li, j, tb:tb + n]
                want = O.decode_attention(qh[li, s, h_n * j:h_n * (j + 1), 0], int(pos_q[s]),
                                          Ck[li, s, j, : nk[li, s, j]], rk[li, j, tb:tb + n], mk[li, j, tb:tb + n],
                                          Cv[li, s, j, : nv[li, s, j]], rv[li, j, tb:tb + n], mv[li, j, tb:tb + n], pos, base)["out"]
                g = got[li, s, h_n * j:h_n * (j + 1)]
                err = np.abs(g - want).max() / np.abs(want).max()
                worst = max(worst, err)
                assert err < tol, (li, s, j, err)
    return worst


@pytest.mark.parametrize("dtype,d,tol", [("bf16", 128, 1e-2), ("f32", 64, 2e-5)])
def test_decode_attention_over_codebooks_of_whole_sequences(dtype, d, tol):
    # CodeBooks over all tokens of two sequences (shallow layers): token t sits at position t; several chunks of 1024
    # tokens and a ragged tail; 4 query heads per KV head
    from paper_2507_06517_b200 import binding as B
    from paper_2507_06517_b200.pipeline import SpindleKVDecodeAttention, SpindleKVPass
    wl = synth.Workload("dec", 2, 2, 8, 2, d, dtype, 8, (2500, 2500), 150, (0.05, 0.3), 4, "gauss", budget_tokens=2500.0, seed=101)
    host = generate(wl)
    p = SpindleKVPass(make_config(wl), wl.seq_lens, torch_dtype(wl))
    K, V = stack_layers(wl, host, [0, 1], "K"), stack_layers(wl, host, [0, 1], "V")
    p.run(K, V, None)
    assert p.device_status()["codebook"][0] == 0
    cbk = {k: v.clone() for k, v in p.cb["K"].items()}
    cbv = {k: v.clone() for k, v in p.cb["V"].items()}
    rng = np.random.default_rng(7)
    q = torch.from_numpy(rng.standard_normal((2, 2, wl.n_q_heads, 1, d)).astype(np.float32)).to(torch_dtype(wl)).cuda()
    pos_q = np.array([2500, 2600], dtype=np.int32)
    att = SpindleKVDecodeAttention(p.cb_batch, wl.n_q_heads, wl.n_kv_heads, d, 4096, rope_base=500000.0)
    out = att.run(q, torch.from_numpy(pos_q).cuda(), cbk, cbv).clone()
    torch.cuda.synchronize()
    _check(wl, out, q, pos_q, cbk, cbv, None, 500000.0, tol)
    again = att.run(q, torch.from_numpy(pos_q).cuda(), cbk, cbv).clone()
    torch.cuda.synchronize()
    assert torch.equal(again, out)                       # fixed summation order: the same bits every time


@pytest.mark.parametrize("d", [128, 64])
def test_decode_attention_for_every_group_size(d):
    # 1, 2, 3, 4 and 8 query heads per KV head: the kernel is unrolled for 1, 2, 4 and 8 (three heads run in the
    # form for four with one slot idle) and sums a token's partial dot products for all heads of the group at once;
    # one chunk plus a ragged second one
    from paper_2507_06517_b200.pipeline import SpindleKVDecodeAttention, SpindleKVPass
    wl = synth.Workload("decg", 1, 1, 16, 2, d, "bf16", 8, (700,), 60, (0.05, 0.3), 4, "gauss", budget_tokens=700.0, seed=103)
    host = generate(wl)
    p = SpindleKVPass(make_config(wl), wl.seq_lens, torch_dtype(wl))
    K, V = stack_layers(wl, host, [0], "K"), stack_layers(wl, host, [0], "V")
    p.run(K, V, None)
    assert p.device_status()["codebook"][0] == 0
    rng = np.random.default_rng(11)
    pos_q = np.array([700], dtype=np.int32)
    for h_n in (1, 2, 3, 4, 8):
        hq = h_n * wl.n_kv_heads
        q = torch.from_numpy(rng.standard_normal((1, 1, hq, 1, d)).astype(np.float32)).to(torch_dtype(wl)).cuda()
        att = SpindleKVDecodeAttention(p.cb_batch, hq, wl.n_kv_heads, d, 1024)
        out = att.run(q, torch.from_numpy(pos_q).cuda(), p.cb["K"], p.cb["V"]).clone()
        torch.cuda.synchronize()
        _check(wl.replace(n_q_heads=hq), out, q, pos_q, p.cb["K"], p.cb["V"], None, 10000.0, 1e-2)


def test_decode_attention_over_an_evicted_and_replaced_cache():
    # the composition as written: every layer keeps k + w tokens (different per layer) and replaces them; the cached
    # tokens keep their original positions (the kept indices), which the rotation must use
    from paper_2507_06517_b200.pipeline import SpindleKVDecodeAttention, SpindleKVLiteralPass
    wl = synth.Workload("declit", 3, -1, 8, 2, 128, "bf16", 32, (1500,), 60, (0.03, 0.3), 2, "recency",
                        budget_tokens=400.0, seed=102)
    layers = list(range(wl.n_layers))
    host = {lam: synth.layer_arrays(wl, lam, need_q=True) for lam in layers}
    K, V, Q = (stack_layers(wl, host, layers, x) for x in ("K", "V", "Q"))
    p = SpindleKVLiteralPass(make_config(wl), wl.seq_lens, torch_dtype(wl))
    p.run(K, V, Q)
    st = p.device_status()
    assert st["evict"][0] == 0 and st["codebook"][0] == 0
    rng = np.random.default_rng(8)
    q = torch.from_numpy(rng.standard_normal((3, 1, wl.n_q_heads, 1, 128)).astype(np.float32)).to(torch.bfloat16).cuda()
    pos_q = np.array([1500], dtype=np.int32)
    # positions of the cached tokens, laid out like the CodeBook call's per-token outputs: [L][H][B * max_keep]
    keep = p.ev.keep_idx[:, :, : p.max_keep].contiguous()
    att = SpindleKVDecodeAttention(p.cb_batch, wl.n_q_heads, wl.n_kv_heads, 128, 2048)
    out = att.run(q, torch.from_numpy(pos_q).cuda(), p.cb["K"], p.cb["V"], positions=keep).clone()
    torch.cuda.synchronize()
    one = wl.replace(seq_lens=(p.max_keep,))
    worst = _check(one, out, q, pos_q, p.cb["K"], p.cb["V"], {"pos": keep.cpu().numpy(), "len": p.kept_host}, 10000.0, 1e-2)
    assert worst > 0.0
    # rotating at the list index instead of the original position gives a different answer: the positions matter
    wrong = att.run(q, torch.from_numpy(pos_q).cuda(), p.cb["K"], p.cb["V"], positions=None).clone()
    torch.cuda.synchronize()
    assert (wrong - out).abs().max() > 1e-2 * out.abs().max()
