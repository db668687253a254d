"""Stand-alone kernels (GEMM, attention, LM head, rollout) against the oracle's arithmetic in fp64."""
import numpy as np
import pytest
import torch

from oracle import model as omodel
from oracle import rollout as orollout
from paper_2509_23094_b200 import binding
from gpu_util import ROW_TOL, row_rel_err

pytestmark = pytest.mark.gpu


def _bf16(shape, seed, std=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(*shape, generator=g) * std).to(torch.bfloat16)


@pytest.mark.parametrize("impl", [1, 2, 0])
@pytest.mark.parametrize("rows,n,N,K", [(200, 200, 256, 128), (300, 131, 384, 256), (128, 128, 128, 64),
                                         (520, 517, 1000, 192), (64, 0, 256, 128), (260, 1, 128, 1024),
                                         (256, 100, 4096, 512), (1024, 130, 2048, 256), (512, 40, 8192, 128),
                                         (300, 290, 1004, 128), (600, 599, 330, 64)])
def test_gemm_matches_fp64(impl, rows, n, N, K):
    A = _bf16((rows, K), 1); W = _bf16((N, K), 2, 0.05); bias = _bf16((N,), 3)
    n_dev = torch.tensor([n], dtype=torch.int32, device="cuda")
    for b in (None, bias):
        Cm = binding.d2c_op_gemm(A.cuda(), W.cuda(), n_dev, bias=None if b is None else b.cuda(), impl=impl)
        torch.cuda.synchronize()
        want = A.double().numpy() @ W.double().numpy().T + (0 if b is None else b.double().numpy())
        got = Cm.float().cpu().numpy()
        assert row_rel_err(got[:n], want[:n]) <= ROW_TOL / 4
        assert np.all(got[n:] == 0)                                   # rows past n_rows are not written


@pytest.mark.parametrize("n", [769, 835, 896, 897, 1023, 1024, 40, 128, 129])
def test_gemm_ragged_row_counts_on_the_pair_kernel(n):
    """Row counts around the 256-row pair tile (one row, 67, 128, 129 and 255 rows in the last tile, and fewer
    rows than one CTA holds) with enough column tiles that the launch keeps full-width tiles and takes no split-K."""
    rows, N, K = 1024, 4864, 128
    A = _bf16((rows, K), 11); W = _bf16((N, K), 12, 0.05); bias = _bf16((N,), 13)
    n_dev = torch.tensor([n], dtype=torch.int32, device="cuda")
    Cm = binding.d2c_op_gemm(A.cuda(), W.cuda(), n_dev, bias=bias.cuda(), impl=0)
    torch.cuda.synchronize()
    want = A.double().numpy()[:n] @ W.double().numpy().T + bias.double().numpy()
    got = Cm.float().cpu().numpy()
    assert row_rel_err(got[:n], want) <= ROW_TOL / 4
    assert np.all(got[n:] == 0)


def _attention_ref(q, kc, vc, row_off, L, Hq, Hkv, Dh):
    rows = q.shape[0]
    o = np.zeros((rows, Hq * Dh)); lse = np.zeros((rows, Hq)); abar = np.zeros((rows, L))
    for b in range(len(row_off) - 1):
        r0, r1 = row_off[b], row_off[b + 1]
        for h in range(Hq):
            g = h // (Hq // Hkv)
            s = q[r0:r1, h * Dh:(h + 1) * Dh] @ kc[b, :L, g].T / np.sqrt(Dh)
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            lse[r0:r1, h] = (m + np.log(e.sum(axis=1, keepdims=True)))[:, 0]
            P = omodel.softmax_rows(s)
            o[r0:r1, h * Dh:(h + 1) * Dh] = P @ vc[b, :L, g]
            abar[r0:r1] += P / Hq
    return o, lse, abar


@pytest.mark.parametrize("impl", [0, 1])
@pytest.mark.parametrize("Hq,Hkv,Dh,L,cache_seq,nbs", [(4, 4, 64, 128, 128, [95]), (4, 2, 64, 200, 256, [1, 130]),
                                                         (4, 1, 128, 333, 400, [64, 0, 65]), (8, 8, 128, 64, 64, [64]),
                                                         (2, 2, 128, 1000, 1024, [129]), (4, 2, 128, 128, 128, [128, 128]),
                                                         (6, 2, 128, 700, 768, [300, 5, 257])])
def test_attention_matches_fp64(impl, Hq, Hkv, Dh, L, cache_seq, nbs):
    B = len(nbs)
    rows = sum(nbs)
    row_off = np.concatenate([[0], np.cumsum(nbs)]).astype(np.int32)
    ldq = (Hq + 2 * Hkv) * Dh                                          # Q sits inside a wider QKV row, as in the step
    q = _bf16((rows + 3, ldq), 5)
    kc = _bf16((B, cache_seq, Hkv, Dh), 6); vc = _bf16((B, cache_seq, Hkv, Dh), 7)
    o, lse, abar = binding.d2c_op_attention(q.cuda(), kc.cuda(), vc.cuda(), torch.from_numpy(row_off).cuda(), L, Hq, Hkv, Dh,
                                            impl=impl)
    torch.cuda.synchronize()
    wo, wl, wa = _attention_ref(q.double().numpy()[:rows], kc.double().numpy(), vc.double().numpy(), row_off, L, Hq, Hkv, Dh)
    assert row_rel_err(o.float().cpu().numpy()[:rows], wo) <= ROW_TOL
    np.testing.assert_allclose(lse.cpu().numpy()[:rows], wl, rtol=0, atol=2e-3)
    got_a = abar.cpu().numpy()[:rows]
    np.testing.assert_allclose(got_a.sum(axis=1), 1.0, atol=1e-4)
    assert row_rel_err(got_a, wa) <= ROW_TOL
    assert np.all(o.float().cpu().numpy()[rows:] == 0)


@pytest.mark.parametrize("rows,n,d,V", [(40, 33, 256, 1024), (130, 129, 128, 1000), (8, 0, 64, 128), (32, 32, 512, 5000)])
def test_lm_head_matches_fp64(rows, n, d, V):
    x = _bf16((rows, d), 8); W = _bf16((V, d), 9, 0.1)
    if V == 1000:                                                      # equal logits: the lower token id must win
        W[777] = W[123]
    n_dev = torch.tensor([n], dtype=torch.int32, device="cuda")
    conf, pred, logits = binding.d2c_op_lm_head(x.cuda(), W.cuda(), n_dev, want_logits=True)
    torch.cuda.synchronize()
    want = x.double().numpy()[:n] @ W.double().numpy().T
    got = logits.cpu().numpy()[:n]
    assert row_rel_err(got, want) <= ROW_TOL / 4
    # the statistics must be exact functions of the logits the kernel itself produced
    g64 = got.astype(np.float64)
    pmax = np.exp(g64 - g64.max(axis=1, keepdims=True)); pmax /= pmax.sum(axis=1, keepdims=True)
    np.testing.assert_array_equal(pred.cpu().numpy()[:n], g64.argmax(axis=1))
    np.testing.assert_allclose(conf.cpu().numpy()[:n], pmax.max(axis=1), rtol=2e-5)
    # and close to the oracle's
    wp = omodel.softmax_rows(want)
    np.testing.assert_allclose(conf.cpu().numpy()[:n], wp.max(axis=1), rtol=5e-2)
    assert np.all(pred.cpu().numpy()[n:] == -1)


@pytest.mark.parametrize("N,B,L,seed", [(1, 1, 64, 0), (3, 2, 200, 1), (5, 3, 333, 2), (2, 1, 1024, 3)])
def test_rollout_matches_chain(N, B, L, seed):
    rng = np.random.default_rng(seed)
    nbs = [int(rng.integers(0, L + 1)) for _ in range(B)]
    if B > 1:
        nbs[1] = 0
    row_off = np.concatenate([[0], np.cumsum(nbs)]).astype(np.int32)
    rows = int(row_off[-1])
    sel = np.concatenate([np.sort(rng.choice(L, nb, replace=False)) for nb in nbs] + [np.zeros(0, int)]).astype(np.int32)
    abar = rng.random((N, max(rows, 1), L)).astype(np.float32) ** 3
    abar /= abar.sum(axis=2, keepdims=True)
    c0 = torch.full((B, L), 7.0, dtype=torch.float32, device="cuda")
    c = binding.d2c_op_rollout(torch.from_numpy(abar).cuda(), torch.from_numpy(np.concatenate([sel, [0]]).astype(np.int32)).cuda(),
                               torch.from_numpy(row_off).cuda(), B, L, c=c0)
    torch.cuda.synchronize()
    got = c.cpu().numpy()
    for b in range(B):
        if nbs[b] == 0:
            assert np.all(got[b] == 7.0)                               # no selected rows: scores stay as they were
            continue
        S = sel[row_off[b]: row_off[b + 1]]
        want = orollout.chain([abar[l, row_off[b]: row_off[b + 1]].astype(np.float64) for l in range(N)], S, L)
        np.testing.assert_allclose(got[b], want, rtol=1e-4, atol=1e-5)
        assert abs(got[b].sum() - L) < 1e-3 * L
