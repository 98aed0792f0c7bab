"""The allocation-free eviction entry point against the ordinary one, through the C ABI.

Some users of the library cannot allocate device memory where the pass runs (an inference server whose
pool owns the whole GPU, a plugin under another framework's allocator lock).  For them
``spindlekv_evict_deep_noalloc`` keeps its scratch in a fixed array inside the library.  It runs the
same kernels, so its outputs must equal the ordinary entry point's bit for bit, also on a second call
that finds the previous call's leftovers in the shared scratch.
"""
import numpy as np
import pytest
import torch

from paper_2507_06517_b200 import synth

from gpu_util import generate, make_config, stack_layers, torch_dtype

pytestmark = pytest.mark.gpu


def _both_ways(wl):
    from paper_2507_06517_b200 import binding as B
    from paper_2507_06517_b200.pipeline import SpindleKVPass
    host = generate(wl)
    deep = list(range(wl.n_shallow, wl.n_layers))
    p = SpindleKVPass(make_config(wl), wl.seq_lens, torch_dtype(wl))
    K = stack_layers(wl, host, deep, "K")
    Q = stack_layers(wl, host, deep, "Q")
    desc = p._desc(K)
    B.spindlekv_evict_deep(p.cfg, p.deep_batch, desc, B.desc_bhnd(Q), p.k_ctx, p.keep_idx, p.keep_cnt, p.scores,
                           p.ws_evict)
    torch.cuda.synchronize()
    want = (p.keep_idx.clone(), p.keep_cnt.clone(), p.scores.clone())
    keep_idx = torch.full_like(p.keep_idx, -7)
    keep_cnt = torch.full_like(p.keep_cnt, -7)
    scores = torch.zeros_like(p.scores)
    B.spindlekv_evict_deep_noalloc(p.cfg, p.deep_batch, desc, B.desc_bhnd(Q), p.k_ctx, keep_idx, keep_cnt, scores)
    torch.cuda.synchronize()
    k = p.k_ctx_host[wl.n_shallow:]
    assert torch.equal(keep_cnt, want[1])
    assert torch.equal(scores, want[2])  # same kernels, same order of operations: identical bits
    for li in range(len(deep)):
        for s, l in enumerate(wl.seq_lens):
            tb = int(synth.cu_seqlens(wl)[s]) if wl.packed else s * wl.max_len
            n = int(k[li, s]) + wl.window
            assert torch.equal(keep_idx[li, :, tb:tb + n], want[0][li, :, tb:tb + n])


def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    _both_ways(synth.workload("C1"))
    wl = synth.Workload("packed", 3, 1, 4, 2, 64, "bf16", 16, (300, 777, 512), 24, (0.05, 0.3), 2, "recency",
                        budget_frac=0.2, seed=12)
    _both_ways(wl)  # second call: the shared scratch still holds the first call's contents
    _both_ways(synth.workload("C1"))


def test_noalloc_rejects_what_does_not_fit():
    # fp32 inputs take the CUDA-core kernels, which keep per-tile row statistics in the scratch: all 16 evicting
    # layers of the 16k-token shape at once need about 34 MB of it.  The rejection comes before any launch.
    from paper_2507_06517_b200 import binding as B
    wl = synth.workload("C3")
    cfg = make_config(wl)
    batch = B.Batch(16, 1, wl.max_len, wl.max_len)
    assert B.spindlekv_workspace_bytes(cfg, batch, B.WS_EVICT) > B.NOALLOC_SCRATCH_BYTES
    t = torch.zeros(64, dtype=torch.float32, device="cuda")
    i = torch.zeros(64, dtype=torch.int32, device="cuda")
    d = B._Tensor(t.data_ptr(), B.F32, 8, 8, 8, 8)
    with pytest.raises(B.SpindleKVError) as e:
        B.spindlekv_evict_deep_noalloc(cfg, batch, d, d, i, i, i, t)
    assert e.value.status == B.WORKSPACE_TOO_SMALL


def test_noalloc_on_the_tensor_core_kernel_and_its_status_word():
    # bf16 with 128 query rows per KV head: the TMA / tensor-core window-score kernel, the only one that writes
    # the device status word.  Its scratch is the status block alone, so a batch that the CUDA-core path could not
    # hold fits; the status word of the call is read back through the NULL form of spindlekv_poll_status.
    from paper_2507_06517_b200 import binding as B
    wl = synth.Workload("noalloc-tc", 2, 0, 32, 8, 128, "bf16", 32, (1500,), 40, (0.05, 0.3), 4, "recency",
                        budget_tokens=300.0, seed=19)
    for _ in range(2):
        _both_ways(wl)
        status, _ = B.spindlekv_poll_status(None)
        assert status == B.OK
    many = wl.replace(n_layers=12, seq_lens=(6000,), budget_tokens=1200.0, name="noalloc-tc-12")   # row statistics of 12 such layers would not fit 8 MiB
    assert B.spindlekv_workspace_bytes(make_config(many), B.Batch(12, 1, 6000, 6000), B.WS_EVICT) > B.NOALLOC_SCRATCH_BYTES
    _both_ways(many)
    assert B.spindlekv_poll_status(None)[0] == B.OK
