"""GPU parity: str_topk_select and str_compact against the oracle's full sort and naive gather.
Integer / byte work: bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_00198_b200 import binding, inputs
from util_gpu import dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.check_status()
    c.close()


@pytest.mark.parametrize("kind", ["uniform", "heavy", "ties", "equal", "ascending", "descending"])
@pytest.mark.parametrize("n,k", [(1, 1), (31, 7), (1000, 250), (1024, 256), (4096, 1024), (5000, 4999),
                                 (32768, 16384), (65536, 6553)])
def test_topk_matches_full_sort(ctx, kind, n, k):
    s = inputs.score_vectors(11, n, kind, batch=2)
    got = binding.str_topk_select(ctx, dev(s), k).cpu().numpy()
    for b in range(2):
        assert np.array_equal(got[b], oracle.topk_select(s[b], k)), (kind, n, k, b)


@pytest.mark.parametrize("kind", ["uniform", "ties", "equal", "descending"])
@pytest.mark.parametrize("n,k,Bz", [(131073, 1000, 1), (200000, 100000, 2), (1048576, 262144, 1), (300001, 300000, 1)])
def test_topk_long_rows_split_over_many_ctas(ctx, kind, n, k, Bz):
    s = inputs.score_vectors(13, n, kind, batch=Bz)
    got = binding.str_topk_select(ctx, dev(s), k).cpu().numpy()
    for b in range(Bz):
        assert np.array_equal(got[b], oracle.topk_select(s[b], k)), (kind, n, k, b)
    if kind == "ties" and Bz == 1:
        # without a workspace the same rows take the one-CTA kernel: same answer
        import ctypes
        out = dev(np.zeros((Bz, k), dtype=np.int32))
        rc = binding.lib().str_topk_select(ctx.handle, Bz, n, k, binding._p(dev(s)), binding._p(out), None, ctypes.c_size_t(0),
                                           binding._stream())
        assert rc == 0 and np.array_equal(out.cpu().numpy(), got)


def test_topk_edge_budgets(ctx):
    s = inputs.score_vectors(12, 777, "uniform", batch=3)
    full = binding.str_topk_select(ctx, dev(s), 777).cpu().numpy()
    assert np.array_equal(full, np.tile(np.arange(777, dtype=np.int32), (3, 1)))     # 100% budget = identity
    assert binding.str_topk_select(ctx, dev(s), 0).shape == (3, 0)
    one = binding.str_topk_select(ctx, dev(s), 1).cpu().numpy()
    assert np.array_equal(one[:, 0], s.argmax(axis=1))
    with pytest.raises(binding.StrError):
        binding.str_topk_select(ctx, dev(s), 778)


def test_topk_negative_and_zero_scores(ctx):
    s = np.array([[0.0, -1.0, 3.0, -0.5, 0.0, 2.0, -7.0, 1e-30]], dtype=np.float32)
    for k in range(9):
        got = binding.str_topk_select(ctx, dev(s), k).cpu().numpy()[0]
        assert np.array_equal(got, oracle.topk_select(s[0], k))


@pytest.mark.parametrize("dtype,D", [("bf16", 4096), ("f32", 256), ("bf16", 8), ("f32", 36)])
@pytest.mark.parametrize("n_vis,n_text,k,Bz", [(1024, 32, 256, 1), (1000, 7, 333, 3), (64, 1, 64, 2), (50, 3, 0, 1)])
def test_compact_is_a_bit_exact_gather(ctx, dtype, D, n_vis, n_text, k, Bz):
    T = n_vis + n_text
    h = inputs.hidden_inputs(21, T, D, dtype, batch=Bz)
    g = inputs.rng(21, 9)
    pos = np.sort(g.choice(10 * T, size=(Bz, T)), axis=1).astype(np.int32)
    idx = g.integers(0, 1 << 30, size=(Bz, T)).astype(np.int32)
    kept = np.stack([np.sort(g.choice(n_vis, size=k, replace=False)) for _ in range(Bz)]).astype(np.int32).reshape(Bz, k)
    ho, po, io = binding.str_compact(ctx, dev(h, dtype), dev(pos), dev(idx), dev(kept), n_text)
    ho = ho.float().cpu().numpy()
    for b in range(Bz):
        rh, rp, ri = oracle.compact(h[b], pos[b], idx[b], kept[b], n_text)
        assert np.array_equal(ho[b], rh) and np.array_equal(po[b].cpu().numpy(), rp)
        assert np.array_equal(io[b].cpu().numpy(), ri)


def test_compact_twice_composes_to_original_ids(ctx):
    n_vis, M, D = 2048, 16, 512
    h = inputs.hidden_inputs(22, n_vis + M, D, "bf16")
    ids = np.arange(n_vis + M, dtype=np.int32)[None]
    g = inputs.rng(22, 9)
    k1 = np.sort(g.choice(n_vis, size=1024, replace=False)).astype(np.int32)[None]
    k2 = np.sort(g.choice(1024, size=512, replace=False)).astype(np.int32)[None]
    h1, p1, i1 = binding.str_compact(ctx, dev(h, "bf16"), dev(ids), dev(ids), dev(k1), M)
    h2, p2, i2 = binding.str_compact(ctx, h1, p1, i1, dev(k2), M)
    i2 = i2.cpu().numpy()[0]
    assert np.array_equal(i2[:512], k1[0][k2[0]]) and np.array_equal(i2[512:], np.arange(n_vis, n_vis + M))
    assert np.array_equal(h2.float().cpu().numpy()[0], h[0][i2]) and np.all(np.diff(p2.cpu().numpy()[0]) > 0)


def test_compact_rejects_bad_arguments(ctx):
    h = dev(inputs.hidden_inputs(23, 10, 8, "f32"))
    with pytest.raises(binding.StrError):       # k > n_vis
        binding.str_compact(ctx, h, None, None, torch.zeros((1, 9), dtype=torch.int32, device="cuda"), 2)
    with pytest.raises(binding.StrError):       # row not a multiple of 16 bytes
        binding.str_compact(ctx, dev(inputs.hidden_inputs(23, 10, 3, "f32")), None, None,
                            torch.zeros((1, 2), dtype=torch.int32, device="cuda"), 2)


@pytest.mark.parametrize("kind", ["uniform", "heavy", "ties", "equal", "ascending"])
@pytest.mark.parametrize("n", [1, 100, 4096, 32768, 100003])
def test_score_density_matches_the_full_sort(ctx, kind, n):
    """Tokens needed for a share of the importance mass (the paper's sparsity statistic), against sort + cumulative sum."""
    s = inputs.score_vectors(44, n, kind, batch=3)
    s[2] = 0.0                                                      # one all-zero row
    for frac in (0.8, 0.5, 1.0):
        got = binding.str_score_density(ctx, dev(s), frac).cpu().numpy()
        for b in range(3):
            want = oracle.score_density(s[b], np.float32(frac))
            if kind in ("ties", "equal"):
                # many equal scores at the threshold: the count of copies still needed is a quotient on the GPU and a
                # running sum in the oracle, which may round differently exactly at a boundary
                assert abs(int(got[b]) - want) <= 1, (kind, n, frac, b)
            else:
                assert int(got[b]) == want, (kind, n, frac, b)
    hot = np.zeros((1, max(n, 2)), dtype=np.float32)
    hot[0, n // 2] = 2.5
    assert int(binding.str_score_density(ctx, dev(hot), 0.8).cpu().numpy()[0]) == 1


def test_bounded_wait_gives_up_and_the_status_word_reports_it_once(ctx):
    """Every pipelined kernel of the library waits on its barriers with a probe limit and, on giving up, records
    STR_ERR_TIMEOUT in the context's status word.  The self-test kernel makes such a wait run out (a barrier that
    nobody signals): the next status check reports the timeout, the one after it is clean, and the context works."""
    ctx.check_status()
    ctx.selftest_wait_timeout(1000)
    with pytest.raises(binding.StrError) as e:
        ctx.check_status()
    assert e.value.code == -5
    ctx.check_status()                                              # cleared by the read
    s = inputs.score_vectors(45, 5000, "uniform")
    kept = binding.str_topk_select(ctx, dev(s), 1250).cpu().numpy()[0]
    assert np.array_equal(kept, oracle.topk_select(s[0], 1250))
    ctx.check_status()


def test_path_counters_tell_tensor_core_from_fallback_calls(ctx):
    """A shape the tensor-core scan tiles and one it does not: the context counts which path each call took."""
    tc0, fb0 = ctx.path_counts()
    d = inputs.ssd_inputs(46, 300, 4, 64, 128, 2, "bf16")
    binding.str_mamba2_prefill(ctx, dev(d["x"], "bf16"), dev(d["dt"]), dev(d["A"]), dev(d["B"], "bf16"), dev(d["C"], "bf16"))
    tc1, fb1 = ctx.path_counts()
    assert (tc1 - tc0, fb1 - fb0) == (1, 0)
    d = inputs.ssd_inputs(46, 300, 4, 16, 32, 2, "f32")
    binding.str_mamba2_prefill(ctx, dev(d["x"]), dev(d["dt"]), dev(d["A"]), dev(d["B"]), dev(d["C"]))
    tc2, fb2 = ctx.path_counts()
    assert (tc2 - tc1, fb2 - fb1) == (0, 1)
    ctx.check_status()
