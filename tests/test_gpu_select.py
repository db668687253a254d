"""Selection kernels against the oracle: index sets, offsets and keys must match bit for bit."""
import numpy as np
import pytest
import torch

from oracle import selection as osel
from paper_2509_23094_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _run_case(B, L, frac_masked, k, p, seed, kind="uniform", ties=0, mode=0, use_key=False, forced=None, sigma=10.0):
    rng = np.random.default_rng(seed)
    mask = (rng.random((B, L)) < frac_masked).astype(np.uint8)
    conf = np.stack([inputs.make_scores(L, seed * 7 + b, "uniform", ties).numpy() for b in range(B)])
    c = np.stack([inputs.make_scores(L, seed * 13 + b, kind, ties).numpy() for b in range(B)])
    okey = np.stack([inputs.make_scores(L, seed * 17 + b, "uniform", ties).numpy() for b in range(B)]) if use_key else None
    f = fo = None
    if forced is not None:
        flat = [x for fb in forced for x in fb]
        f = torch.tensor(flat if flat else [0], dtype=torch.int32, device="cuda")
        fo = torch.tensor(np.cumsum([0] + [len(fb) for fb in forced]), dtype=torch.int32, device="cuda")
    out = binding.d2c_op_select(torch.from_numpy(mask).cuda(), torch.from_numpy(conf).cuda(), torch.from_numpy(c).cuda(),
                                k, p, sigma=sigma, stage2_candidates=mode,
                                override_key=None if okey is None else torch.from_numpy(okey).cuda(), forced=f, forced_off=fo)
    torch.cuda.synchronize()
    ro = out["row_off"].cpu().numpy(); sel = out["sel_idx"].cpu().numpy()
    lmo = out["lm_off"].cpu().numpy(); lmr = out["lm_rows"].cpu().numpy()
    slot = out["slot_of_pos"].cpu().numpy(); key = out["key"].cpu().numpy()
    assert ro[0] == 0 and lmo[0] == 0
    for b in range(B):
        S, m_star, u = osel.select_rows(mask[b], conf[b], c[b], k, p, sigma, forced=(forced[b] if forced else ()),
                                        stage2_candidates=mode, key=None if okey is None else okey[b])
        got = sel[ro[b]: ro[b + 1]]
        np.testing.assert_array_equal(got, S, err_msg=f"seq {b}")
        if okey is None:
            want_key = osel.stage1_keys(mask[b], conf[b], sigma)
            np.testing.assert_array_equal(key[b].view(np.uint32), want_key.view(np.uint32))
        # rows that go through the LM head: selected and masked, as global row numbers in ascending order
        want_lm = [ro[b] + i for i, pos in enumerate(S) if mask[b, pos]]
        np.testing.assert_array_equal(lmr[lmo[b]: lmo[b + 1]], want_lm)
        want_slot = np.full(L, -1); want_slot[S] = ro[b] + np.arange(len(S))
        np.testing.assert_array_equal(slot[b], want_slot)


@pytest.mark.parametrize("seed", range(6))
def test_random_cases(seed):
    rng = np.random.default_rng(1000 + seed)
    B = int(rng.integers(1, 4)); L = int(rng.integers(1, 700))
    _run_case(B, L, float(rng.random()), int(rng.integers(0, 40)), float(rng.random()), seed,
              kind=["uniform", "zipf", "flat"][seed % 3], ties=[0, 16, 3][seed % 3], mode=seed % 2)


@pytest.mark.parametrize("L", [1, 31, 32, 33, 127, 128, 129, 600, 1024, 1025, 2048, 4096, 5000, 8192])
def test_sizes_around_tile_boundaries(L):
    _run_case(2, L, 0.3, 32, 0.9, L, kind="flat")
    _run_case(1, L, 0.5, 8, 0.1, L + 1, kind="zipf", use_key=True)


def test_degenerate_cases():
    _run_case(2, 200, 0.4, 0, 0.0, 1)                    # nothing selected
    _run_case(2, 200, 0.4, 10 ** 6, 1.0, 2)              # everything selected
    _run_case(2, 200, 0.4, 10 ** 6, 2.0, 3, mode=1)
    _run_case(2, 200, 0.0, 5, 0.5, 4)                    # nothing masked
    _run_case(2, 200, 1.0, 5, 0.5, 5)                    # everything masked: no candidates in mode 0
    _run_case(2, 200, 1.0, 5, 0.5, 6, mode=1)
    _run_case(1, 300, 0.3, 4, 0.25, 7, ties=2)           # heavy ties
    _run_case(2, 64, 0.5, 3, 0.2, 8, forced=[[0, 63, 5, 5], []])
    _run_case(1, 500, 0.3, 16, 0.5, 9, sigma=3.0)
    _run_case(1, 500, 0.3, 16, 0.5, 10, sigma=40.0)
    _run_case(1, 300, 0.3, 4, 1.0 - 2.0 ** -24, 11)


def test_bad_scores_count_as_zero():
    L = 100
    mask = np.zeros((1, L), dtype=np.uint8); mask[0, 50:60] = 1
    conf = np.full((1, L), 0.5, dtype=np.float32); conf[0, 52] = np.nan; conf[0, 53] = -1.0
    c = np.linspace(0, 1, L, dtype=np.float32)[None].copy(); c[0, 3] = np.nan; c[0, 4] = -5.0; c[0, 5] = np.inf
    out = binding.d2c_op_select(torch.from_numpy(mask).cuda(), torch.from_numpy(conf).cuda(), torch.from_numpy(c).cuda(), 9, 0.5)
    ro = out["row_off"].cpu().numpy(); sel = out["sel_idx"].cpu().numpy()[: ro[1]]
    S, _, _ = osel.select_rows(mask[0], conf[0], c[0], 9, 0.5, 10.0)
    np.testing.assert_array_equal(sel, S)


def test_full_size_workload_patterns():
    """The mask patterns and sizes of the five workloads, with peaked and flat scores."""
    for name, wl in inputs.WORKLOADS.items():
        mask = inputs.make_mask(wl).numpy()
        B, L = mask.shape
        for kind, p in (("flat", wl.p), ("zipf", 0.1)):
            conf = np.stack([inputs.make_scores(L, 31 + b, "uniform").numpy() for b in range(B)])
            c = np.stack([inputs.make_scores(L, 57 + b, kind).numpy() for b in range(B)])
            out = binding.d2c_op_select(torch.from_numpy(mask).cuda(), torch.from_numpy(conf).cuda(),
                                        torch.from_numpy(c).cuda(), wl.k, p, sigma=wl.sigma)
            ro = out["row_off"].cpu().numpy(); sel = out["sel_idx"].cpu().numpy()
            for b in range(B):
                S, m_star, _ = osel.select_rows(mask[b], conf[b], c[b], wl.k, p, wl.sigma)
                np.testing.assert_array_equal(sel[ro[b]: ro[b + 1]], S, err_msg=f"{name} seq {b}")
                assert len(m_star) == min(wl.k, int(mask[b].sum()))
