"""GPU parity of the split-K forward over a paged K/V pool with one length per sequence.

The function per sequence is plain attention over that sequence's keys, so the
oracle is ``attn_naive`` on the keys gathered (on the CPU, by the test) from the
pool in table order; nothing of the method lives in the gathering."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2505_14201_b200 import synth

pytestmark = pytest.mark.gpu

BF16_MAX, BF16_MEAN = 1e-2, 1e-3


def f32_scale(d):
    return float(np.float32(1.0 / math.sqrt(d)))


def build_pool(lens, H, d, page_size, seed, spare=3):
    """Seeded K/V for every sequence, scattered over a shuffled page pool.
    Returns (k_pages, v_pages, block_table, seq_lens, per-sequence contiguous K, V)."""
    g = torch.Generator().manual_seed(seed)
    B = len(lens)
    max_pages = max(1, max((n + page_size - 1) // page_size for n in lens))
    need = sum((n + page_size - 1) // page_size for n in lens)
    num_pages = need + spare
    order = torch.randperm(num_pages, generator=g).tolist()
    # unowned pages and page tails hold large garbage: a wrong address shows up in the result
    k_pages = (torch.randn(num_pages, H, page_size, d, generator=g) * 30).to(torch.bfloat16)
    v_pages = (torch.randn(num_pages, H, page_size, d, generator=g) * 30).to(torch.bfloat16)
    table = torch.full((B, max_pages), -1, dtype=torch.int32)
    ks, vs = [], []
    nxt = 0
    for b, n in enumerate(lens):
        _, k, v = synth.random_qkv(1, H, 1, max(n, 1), d, seed=seed * 100 + b)
        k, v = k[0, :, :n], v[0, :, :n]
        ks.append(k); vs.append(v)
        for p in range((n + page_size - 1) // page_size):
            page = order[nxt]; nxt += 1
            table[b, p] = page
            m = min(page_size, n - p * page_size)
            k_pages[page, :, :m] = k[:, p * page_size:p * page_size + m]
            v_pages[page, :, :m] = v[:, p * page_size:p * page_size + m]
    return k_pages, v_pages, table, torch.tensor(lens, dtype=torch.int32), ks, vs


def check(got, q, ks, vs, lens, sc, what):
    B, H, Nq, d = q.shape
    for b in range(B):
        if lens[b] == 0:
            assert torch.all(got[b] == 0), (what, b, "empty sequence must give 0")
            continue
        want = oracle.attn_naive(q[b:b + 1], ks[b][None], vs[b][None], sc, False)
        err = np.abs(got[b:b + 1].double().cpu().numpy() - want)
        assert np.all(np.isfinite(got[b].float().cpu().numpy())), (what, b)
        assert err.max() <= BF16_MAX, (what, b, lens[b], err.max())
        assert err.mean() <= BF16_MEAN, (what, b, lens[b], err.mean())


@pytest.mark.parametrize("d,page_size,lens,H,Nq,splits", [
    (128, 64, [1, 63, 64, 65, 1000, 4097], 3, 1, 0),
    (128, 128, [300, 0, 2048, 5], 2, 1, 4),
    (128, 256, [9000, 17, 4096], 4, 2, 7),       # two query rows per head, splits that are empty for short sequences
    (64, 128, [1, 127, 128, 129, 3000], 3, 1, 0),
    (64, 256, [6000, 250], 5, 3, 3),
    (128, 64, [40000], 2, 1, 0),                 # more work items than fit in one pass of a few CTAs, long sequence
])
def test_paged_matches_oracle(flashd_lib, d, page_size, lens, H, Nq, splits):
    sc = f32_scale(d)
    k_pages, v_pages, table, seq_lens, ks, vs = build_pool(lens, H, d, page_size, seed=7 + d + page_size)
    q, _, _ = synth.random_qkv(len(lens), H, Nq, 1, d, seed=99)
    got = flashd_lib.flashd_attn_fwd_splitk_paged(q.cuda(), k_pages.cuda(), v_pages.cuda(), table.cuda(),
                                                  seq_lens.cuda(), sc, splits)
    st, detail = flashd_lib.flashd_last_device_status()
    assert st == 0, detail
    check(got, q, ks, vs, lens, sc, (d, page_size))


def test_paged_equals_contiguous_kernel(flashd_lib):
    """Equal lengths that are a multiple of split x ring stage: the ranges of the paged and the
    contiguous kernel coincide, and so must the results, bit for bit."""
    d, H, B, n, page_size, S = 128, 3, 2, 4096, 128, 4
    k_pages, v_pages, table, seq_lens, ks, vs = build_pool([n] * B, H, d, page_size, seed=5)
    q, _, _ = synth.random_qkv(B, H, 1, 1, d, seed=6)
    sc = f32_scale(d)
    paged = flashd_lib.flashd_attn_fwd_splitk_paged(q.cuda(), k_pages.cuda(), v_pages.cuda(), table.cuda(),
                                                    seq_lens.cuda(), sc, S)
    k = torch.stack(ks).contiguous()
    v = torch.stack(vs).contiguous()
    flat = flashd_lib.flashd_attn_fwd_splitk(q.cuda(), k.cuda(), v.cuda(), sc, S)
    assert torch.equal(paged.view(torch.int16), flat.view(torch.int16))


def test_bad_table_is_reported_not_followed(flashd_lib):
    """A page index outside the pool and a length the table cannot hold are flagged in the
    device status word; the kernel finishes and reads nothing outside the pool."""
    d, H, page_size = 128, 2, 64
    k_pages, v_pages, table, seq_lens, ks, vs = build_pool([200, 100], H, d, page_size, seed=11)
    q, _, _ = synth.random_qkv(2, H, 1, 1, d, seed=12)
    sc = f32_scale(d)
    bad = table.clone(); bad[0, 1] = k_pages.shape[0] + 5
    flashd_lib.flashd_attn_fwd_splitk_paged(q.cuda(), k_pages.cuda(), v_pages.cuda(), bad.cuda(), seq_lens.cuda(), sc, 2)
    st, detail = flashd_lib.flashd_last_device_status()
    assert st == 2, (st, detail)                 # FLASHD_ERR_SHAPE
    long = seq_lens.clone(); long[1] = table.shape[1] * page_size + 1
    flashd_lib.flashd_attn_fwd_splitk_paged(q.cuda(), k_pages.cuda(), v_pages.cuda(), table.cuda(), long.cuda(), sc, 2)
    st, detail = flashd_lib.flashd_last_device_status()
    assert st == 2, (st, detail)
    # the status word is cleared by the read: a good call is clean again and right
    got = flashd_lib.flashd_attn_fwd_splitk_paged(q.cuda(), k_pages.cuda(), v_pages.cuda(), table.cuda(), seq_lens.cuda(), sc, 2)
    st, detail = flashd_lib.flashd_last_device_status()
    assert st == 0, detail
    check(got, q, ks, vs, [200, 100], sc, "after bad tables")


@pytest.mark.parametrize("d,page_size,lens,H,Nq,splits", [
    (128, 128, [1, 127, 128, 129, 3000], 3, 1, 0),
    (128, 256, [5000, 0, 600], 2, 2, 3),
    (64, 256, [255, 256, 257, 2000], 3, 1, 0),
])
def test_paged_fp8_pool_matches_oracle(flashd_lib, d, page_size, lens, H, Nq, splits):
    """The pool stored as FP8-E4M3: the oracle takes the stored values widened exactly."""
    F8 = torch.float8_e4m3fn
    sc = f32_scale(d)
    k_pages, v_pages, table, seq_lens, ks, vs = build_pool(lens, H, d, page_size, seed=3 + d + page_size)
    k_pages = (k_pages.float() / 30).to(F8)       # the garbage of unowned pages stays large against the keys
    v_pages = (v_pages.float() / 30).to(F8)
    ks = [x.to(F8) for x in ks]
    vs = [x.to(F8) for x in vs]
    # owned keys must be the E4M3 rounding of the sequences' keys, whatever the pool held before
    for b, n in enumerate(lens):
        for p in range((n + page_size - 1) // page_size):
            m = min(page_size, n - p * page_size)
            k_pages[table[b, p], :, :m] = ks[b][:, p * page_size:p * page_size + m]
            v_pages[table[b, p], :, :m] = vs[b][:, p * page_size:p * page_size + m]
    q, _, _ = synth.random_qkv(len(lens), H, Nq, 1, d, seed=98)
    got = flashd_lib.flashd_attn_fwd_splitk_paged(q.cuda(), k_pages.cuda(), v_pages.cuda(), table.cuda(),
                                                  seq_lens.cuda(), sc, splits)
    st, detail = flashd_lib.flashd_last_device_status()
    assert st == 0, detail
    check(got, q, ks, vs, lens, sc, ("fp8", d, page_size))


@pytest.mark.parametrize("d,page_size,lens,Hkv,G,Nq,causal,splits", [
    (128, 128, [1, 127, 128, 129, 3000], 2, 4, 1, False, 0),
    (128, 256, [5000, 0, 600, 255], 2, 8, 1, False, 3),
    (128, 128, [2, 131, 1000], 3, 2, 2, True, 0),          # two positions per head, causal among themselves
    (64, 128, [1, 128, 129, 2000], 2, 4, 2, True, 2),
    (64, 256, [4100, 77], 1, 7, 1, False, 0),
])
def test_paged_grouped_query_matches_oracle(flashd_lib, d, page_size, lens, Hkv, G, Nq, causal, splits):
    """G query heads per K/V head over the paged pool; page tails past a sequence's end hold NaN,
    which must not reach the output (their weights are zero and their V entries are cleared)."""
    sc = f32_scale(d)
    k_pages, v_pages, table, seq_lens, ks, vs = build_pool(lens, Hkv, d, page_size, seed=21 + d + page_size + G)
    nan = torch.tensor(float("nan"), dtype=torch.bfloat16)
    for b, n in enumerate(lens):
        if n % page_size:
            last = table[b, (n - 1) // page_size]
            k_pages[last, :, n % page_size:] = nan
            v_pages[last, :, n % page_size:] = nan
    B = len(lens)
    q, _, _ = synth.random_qkv(B, Hkv * G, Nq, 1, d, seed=97)
    got = flashd_lib.flashd_attn_fwd_gqa_paged(q.cuda(), k_pages.cuda(), v_pages.cuda(), table.cuda(),
                                               seq_lens.cuda(), sc, splits, causal=causal)
    st, detail = flashd_lib.flashd_last_device_status()
    assert st == 0, detail
    g = got.cpu()
    assert torch.all(torch.isfinite(g.float()))
    errs = []
    for b, n in enumerate(lens):
        for iq in range(Nq):
            vis = n - Nq + iq + 1 if causal else n      # keys visible to this position
            if vis <= 0:
                assert torch.all(g[b, :, iq] == 0), (b, iq)
                continue
            kk = ks[b][:, :vis].repeat_interleave(G, dim=0)[None]
            vv = vs[b][:, :vis].repeat_interleave(G, dim=0)[None]
            want = oracle.attn_naive(q[b:b + 1, :, iq:iq + 1], kk, vv, sc, False)
            err = np.abs(g[b:b + 1, :, iq:iq + 1].double().numpy() - want)
            # the bf16 output grid is coarser than the bound above 2 in magnitude: half an ulp is 2^-9 |o|
            assert np.all(err <= BF16_MAX + 2.0 ** -9 * np.abs(want)), (b, iq, n, err.max())
            errs.append(err.ravel())
    # the mean bound is a statement about a workload, not about a two-key sequence: taken over the batch
    assert np.concatenate(errs).mean() <= BF16_MEAN
