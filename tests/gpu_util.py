"""Helpers for the GPU parity tests: run the library through its C ABI and apply the acceptance rules."""
from __future__ import annotations

import numpy as np
import torch

from oracle import oracle_topk
from oracle.acceptance import REL_TOL, canonical_topk_of, check_row_indices, check_row_scores
from paper_2607_11976_b200 import binding as lt


def run_topk(inp, tunables=None, entry="ex"):
    """Returns (idx [T,k] int32, score [T,k] fp32, status[8]) as numpy arrays."""
    q, w, k, ks = lt.to_device(inp)
    out_idx = torch.full((inp.T, inp.topk), -7, dtype=torch.int32, device="cuda")
    out_score = torch.full((inp.T, inp.topk), float("nan"), dtype=torch.float32, device="cuda")
    if entry == "13":
        lt.lt_indexer_topk(q, w, k, ks, inp.topk, inp.causal_offset, out_idx, out_score)
        status = lt.lt_read_status(None)
    else:
        ws = lt.alloc_workspace(inp.dtype, inp.T, inp.N, inp.H, inp.D, inp.topk, tunables)
        lt.lt_indexer_topk_ex(inp.dtype, q, w, k, ks, inp.topk, inp.causal_offset, out_idx, out_score, ws, tunables)
        status = lt.lt_read_status(ws)
    torch.cuda.synchronize()
    # only the bounds-checking build can set this bit (the whole suite also runs against it: LT_INDEXER_LIB)
    assert status[0] & lt.LT_STATUS_BOUNDS == 0, "an index check of the bounds-checking build failed"
    return out_idx.cpu().numpy(), out_score.cpu().numpy(), status


def run_unfused(inp, rows_per_pass=64, path=lt.LT_PATH_AUTO):
    q, w, k, ks = lt.to_device(inp)
    out_idx = torch.full((inp.T, inp.topk), -7, dtype=torch.int32, device="cuda")
    out_score = torch.full((inp.T, inp.topk), float("nan"), dtype=torch.float32, device="cuda")
    buf = torch.empty(256 + rows_per_pass * inp.N * 4, dtype=torch.uint8, device="cuda")
    lt.lt_unfused_topk(inp.dtype, q, w, k, ks, inp.topk, inp.causal_offset, out_idx, out_score, buf, path)
    status = lt.lt_read_status(buf)
    assert status[0] & lt.LT_STATUS_BOUNDS == 0, "an index check of the bounds-checking build failed"
    return out_idx.cpu().numpy(), out_score.cpu().numpy(), status


def dump_scores(inp, row_begin, row_end, path=lt.LT_PATH_AUTO):
    q, w, k, ks = lt.to_device(inp)
    out = torch.full((row_end - row_begin, inp.N), float("nan"), dtype=torch.float32, device="cuda")
    lt.lt_indexer_scores(inp.dtype, q, w, k, ks, inp.causal_offset, row_begin, row_end, out, path)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def assert_matches_oracle(inp, idx, score, rows, dumped=None, dumped_row0=0):
    """Index rule + score rule against the oracle for `rows`; if `dumped` (the library's own dense
    scores, row r of it = row dumped_row0 + r) is given, also the bit-exact own-scores rule."""
    ora = oracle_topk(inp, rows=rows, keep_scores=True)
    worst = 0.0
    swaps = 0
    for r, t in enumerate(ora.rows):
        t = int(t)
        full = ora.full[r]
        tol = REL_TOL * ora.rms[r]
        ok, msg = check_row_indices(idx[t].astype(np.int64), ora.idx[r], full, ora.kth[r], tol)
        assert ok, f"row {t}: {msg}"
        swaps += int(msg.split()[0])
        sel = idx[t][idx[t] >= 0]
        err = np.abs(score[t][: sel.shape[0]].astype(np.float64) - full[sel]).max() if sel.size else 0.0
        assert err <= tol, f"row {t}: selected score error {err:.3e} > tol {tol:.3e}"
        worst = max(worst, err / tol if tol > 0 else 0.0)
        assert np.all(np.isneginf(score[t][sel.shape[0]:])), f"row {t}: padding scores are not -inf"
        if dumped is not None:
            d = dumped[t - dumped_row0]
            n_vis = full.shape[0]
            ok_s, derr = check_row_scores(d, full, tol)
            assert ok_s, f"row {t}: dumped score error {derr:.3e} > tol {tol:.3e}, or a masked key is not -inf"
            want_idx, want_val = canonical_topk_of(d, n_vis, inp.topk)
            assert np.array_equal(idx[t].astype(np.int64), want_idx), f"row {t}: not the exact top-k of the library's own scores"
            assert np.array_equal(score[t].view(np.uint32), want_val.view(np.uint32)), f"row {t}: out_score bits differ from the dump"
    return worst, swaps


def assert_own_scores_rule(inp, idx, score, dumped, rows, dumped_row0=0):
    """Bit-exact: idx/score are the (score desc, index asc) top-k of the library's own dump."""
    for t in rows:
        n_vis = inp.visible(int(t))
        want_idx, want_val = canonical_topk_of(dumped[t - dumped_row0], n_vis, inp.topk)
        assert np.array_equal(idx[t].astype(np.int64), want_idx), f"row {t}: not the exact top-k of the library's own scores"
        assert np.array_equal(score[t].view(np.uint32), want_val.view(np.uint32)), f"row {t}: out_score bits differ"
