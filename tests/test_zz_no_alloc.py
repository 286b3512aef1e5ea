"""The allocation-free pair sampler against the ordinary one.

Some users of the library cannot allocate device memory when they need the pair list (all of
it is already handed out, or allocation is forbidden after start-up), so the library offers
`w2v_sample_pairs_noalloc`, which works entirely inside a fixed array that ships with the
library.  This test drives both entry points through the C ABI on the same inputs and expects
identical index lists and counters -- twice in a row with different chunks, because the fixed
array keeps the previous call's contents and nothing stale may leak into the next result.
It is collected last on purpose, and passes alone in a fresh process as well as after the rest.
"""
import numpy as np
import pytest
import torch

from paper_1606_08495_b200 import binding, corpus

pytestmark = pytest.mark.gpu

MAX_TOKENS = 65536


def both_ways(model, toks, W, N):
    t = torch.from_numpy(np.ascontiguousarray(toks, dtype=np.int32)).cuda()
    n = t.numel()
    cap = max(1, n * 2 * W)
    outs = []
    for fn in (binding.w2v_sample_pairs, binding.w2v_sample_pairs_noalloc):
        centre = torch.full((cap,), -7, dtype=torch.int32, device="cuda")
        context = torch.full((cap,), -7, dtype=torch.int32, device="cuda")
        negs = torch.full((cap * N,), -7, dtype=torch.int32, device="cuda")
        st = binding.StepStats()
        rc, P = fn(model.h, t, n, W, N, centre, context, negs, cap, st)
        assert rc == binding.W2V_OK
        outs.append((P, centre[:P].cpu().numpy(), context[:P].cpu().numpy(),
                     negs[: P * N].cpu().numpy(), st.as_dict()))
    return outs


def test_noalloc_sampler_matches_the_ordinary_one_twice_in_a_row():
    cfg = corpus.scaled(corpus.CONFIGS["small"], d=8)
    cp = corpus.Corpus(cfg)
    model = binding.W2V(cfg["vocab"], cfg["d"], seed=5)
    model.build_alias(cp.counts, cfg["subsample_t"])
    W, N = cfg["window"], cfg["negatives"]
    # first a large chunk, then a smaller one with another step number: whatever the first call
    # left behind in the fixed array must not show up in the second result
    # the third chunk is small enough for the ordinary call's one-launch sampler (at most 8192 tokens),
    # which the allocation-free call never uses: two different kernel sequences, one answer
    for step, words in ((0, 60_000), (3, 9_000), (4, 5_000)):
        model.set_step(step)
        toks = cp.chunk(step, words)
        assert len(toks) <= MAX_TOKENS
        ref, got = both_ways(model, toks, W, N)
        assert ref[0] == got[0] and ref[0] > 1000
        for a, b in zip(ref[1:4], got[1:4]):
            assert np.array_equal(a, b)
        assert ref[4] == got[4]
    model.close()


def test_noalloc_sampler_empty_chunk_and_ids_outside_the_vocabulary():
    model = binding.W2V(50, 8, seed=2)
    model.build_alias(np.full(50, 4, dtype=np.uint64), 0.0)
    t = torch.zeros(1, dtype=torch.int32, device="cuda")
    for fn in (binding.w2v_sample_pairs, binding.w2v_sample_pairs_noalloc):
        st = binding.StepStats()
        rc, P = fn(model.h, t, 0, 3, 2, None, None, None, 0, st)           # n = 0
        assert rc == binding.W2V_OK and P == 0 and st.kept == 0 and st.pairs == 0
    toks = np.array([1, 2, 50, 3, -1, 4, -5, 6, 7, -1, 9], dtype=np.int32)  # 50 and -5 are not word ids
    t = torch.from_numpy(toks).cuda()
    cap = len(toks) * 6
    res = []
    for fn in (binding.w2v_sample_pairs, binding.w2v_sample_pairs_noalloc):
        centre = torch.full((cap,), -7, dtype=torch.int32, device="cuda")
        context = torch.full((cap,), -7, dtype=torch.int32, device="cuda")
        negs = torch.full((cap * 2,), -7, dtype=torch.int32, device="cuda")
        st = binding.StepStats()
        rc, P = fn(model.h, t, len(toks), 3, 2, centre, context, negs, cap, st, allow=(binding.W2V_ERR_TOKEN_RANGE,))
        assert rc == binding.W2V_ERR_TOKEN_RANGE and st.oov == 2 and (st.status & 1)
        res.append((P, centre[:P].tolist(), context[:P].tolist(), negs[: 2 * P].tolist(), st.as_dict()))
    assert res[0] == res[1] and res[0][0] > 0
    model.close()


def test_noalloc_sampler_refuses_chunks_beyond_its_fixed_scratch():
    model = binding.W2V(100, 8, seed=1)
    model.build_alias(np.full(100, 3, dtype=np.uint64), 0.0)
    t = torch.zeros(MAX_TOKENS + 1, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.W2VError) as e:
        binding.w2v_sample_pairs_noalloc(model.h, t, t.numel(), 2, 2, None, None, None, 0)
    assert e.value.code == binding.W2V_ERR_CAPACITY and "65536" in str(e.value)
    # exactly the maximum is served
    st = binding.StepStats()
    rc, P = binding.w2v_sample_pairs_noalloc(model.h, t[:MAX_TOKENS], MAX_TOKENS, 2, 2, None, None, None, 0, st,
                                             allow=(binding.W2V_ERR_CAPACITY,))
    assert P == st.pairs and st.kept == MAX_TOKENS
    model.close()
