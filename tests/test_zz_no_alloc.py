"""The allocation-free acceptance entry point against the regular one (GPU, through the C ABI).

Some callers cannot allocate device memory at the moment they need an acceptance walk - a
latency-critical serving loop that must not trigger the implicit synchronisation of an allocation, a
process whose memory is owned by another allocator (a caching pool, a fixed arena), where a library's
own cudaMalloc would fail or take memory that allocator counts on.  For them
``ssd_accept_tree_noalloc`` keeps its scratch in fixed device arrays of the library.  The results are
compared with the regular entry point AND with the CPU oracle (the single-CTA walk kernel behind this
entry point is not reached by any other test), and the free device memory is checked not to move across
the calls.  This file is named so that pytest collects it last: if it fails, every other test has
already run.  It passes both alone in a fresh process and after the rest of the suite.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import ssd_synth
from oracle import ssd_oracle

pytestmark = pytest.mark.gpu


def _call_regular(ssd, ctx, lg, dp, tokens, parent, mode, seed, step, T, k):
    rng = ssd.binding.ssd_rng(seed, step)
    path, nxt = ctx.accept_tree(lg.data_ptr(), dp.data_ptr() if dp is not None else None, tokens, parent, mode=mode,
                                temperature=T, top_k=k, rng=rng)
    return path, nxt, rng.step


def _call_noalloc(ssd, lg, dp, tokens, parent, V, mode, seed, step, T, k):
    lib = ssd.lib()
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    n = len(tokens)
    samp = ssd.binding.ssd_sampling(mode, T, k)
    rng = ssd.binding.ssd_rng(seed, step)
    path = np.zeros(n, dtype=np.int32)
    n_path, nxt = C.c_int32(0), C.c_int32(-1)
    rc = lib.ssd_accept_tree_noalloc(0, C.c_void_p(torch.cuda.current_stream().cuda_stream), C.c_void_p(lg.data_ptr()),
                                     C.c_void_p(dp.data_ptr() if dp is not None else 0), tokens.ctypes.data, parent.ctypes.data,
                                     n, V, C.byref(samp), C.byref(rng), path.ctypes.data, C.byref(n_path), C.byref(nxt))
    return rc, [int(v) for v in path[:n_path.value]], int(nxt.value), rng.step


@pytest.mark.parametrize("V", [1024, 50257])
def test_noalloc_entry_point_matches_regular_entry_point_twice_in_a_row(V):
    import paper_2308_04623_b200 as ssd
    cfg = ssd_synth.config("tiny", vocab=V)
    ctx = ssd.Context(cfg, device=0, stream=torch.cuda.current_stream().cuda_stream)  # regular entry point needs a context
    try:
        rng = np.random.default_rng(V)
        parent = ssd_synth.tree_branching(24, (3, 2, 2, 1, 1))
        n = len(parent)
        calls = fragile = 0
        for rep in range(2):  # two calls in a row per setting: the shared scratch keeps the previous call's contents
            logits = (rng.normal(size=(n, V)) * 2.5).astype(np.float32)
            probs = np.exp(logits.astype(np.float64))
            probs /= probs.sum(axis=1, keepdims=True)
            draft = np.zeros((n, V), dtype=np.float32)
            tokens = np.zeros(n, dtype=np.int32)
            for c in range(1, n):
                mix = 0.7 * probs[parent[c]] + 0.3 * rng.dirichlet(np.full(V, 0.5))
                draft[c] = mix.astype(np.float32)
                tokens[c] = rng.choice(V, p=mix / mix.sum())
            lg = torch.from_numpy(logits).cuda()
            dp = torch.from_numpy(draft).cuda()
            # one warm call (symbol look-up, lazy module load), then the free device memory must not move
            # (the regular entry point is warmed too: it grows its own per-context scratch on its first sampling call)
            _call_noalloc(ssd, lg, dp, tokens, parent, V, ssd.SSD_SAMPLING, 1, 0, 1.0, 0)
            _call_noalloc(ssd, lg, dp, tokens, parent, V, ssd.SSD_GREEDY, 1, 0, 1.0, 0)
            _call_regular(ssd, ctx, lg, dp, tokens, parent, ssd.SSD_SAMPLING, 1, 0, 1.0, 50)
            _call_regular(ssd, ctx, lg, dp, tokens, parent, ssd.SSD_GREEDY, 1, 0, 1.0, 0)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            for mode, T, k in ((ssd.SSD_GREEDY, 1.0, 0), (ssd.SSD_SAMPLING, 1.0, 0), (ssd.SSD_SAMPLING, 0.75, 50)):
                for step in range(6):
                    want = _call_regular(ssd, ctx, lg, dp, tokens, parent, mode, 11, step, T, k)
                    rc, path, nxt, new_step = _call_noalloc(ssd, lg, dp, tokens, parent, V, mode, 11, step, T, k)
                    assert rc == ssd.SSD_OK
                    assert (path, nxt, new_step) == want  # integer results: exact
                    opath, onxt, margin = ssd_oracle.accept_tree(logits, draft if mode else None, tokens, parent, mode=mode,
                                                                 temperature=float(np.float32(T)), top_k=k, seed=11, step=step)
                    if (path, nxt) != (opath, onxt):
                        assert margin < 1e-9, (mode, T, k, step, margin)
                        fragile += 1
                    calls += 1
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before  # nothing was allocated on the device
        assert calls == 36
        assert fragile == 0
    finally:
        ctx.close()


def test_noalloc_entry_point_refuses_sizes_beyond_its_fixed_scratch():
    import paper_2308_04623_b200 as ssd
    V = 65536 + 1
    lg = torch.zeros((2, 8), dtype=torch.float32, device="cuda")  # never read: the size check comes first
    rc, path, nxt, step = _call_noalloc(ssd, lg, None, [0, 1], [-1, 0], V, ssd.SSD_GREEDY, 0, 0, 1.0, 0)
    assert rc == ssd.SSD_ERR_UNSUPPORTED and step == 0
    rc, *_ = _call_noalloc(ssd, lg, None, [0] * 257, [-1] + list(range(256)), 8, ssd.SSD_GREEDY, 0, 0, 1.0, 0)
    assert rc == ssd.SSD_ERR_INVALID_TREE
    rc, *_ = _call_noalloc(ssd, lg, None, [0, 1], [-1, 0], 8, ssd.SSD_SAMPLING, 0, 0, 1.0, 0)  # sampling without draft rows
    assert rc == ssd.SSD_ERR_BAD_ARG
