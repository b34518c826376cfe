"""Acceptance rule for GPU results against the CPU oracle.

Times: within 1e-12 relative.  Integer picks (strategy id, segment size): equal to the oracle's
wherever the oracle's runner-up is more than 1e-9 (relative) behind its best; inside that margin
the GPU may pick another candidate, provided the oracle's own time for that candidate is within
1e-9 of the oracle's best and the GPU's reported time matches the oracle's time for that
candidate to 1e-12.
"""
from __future__ import annotations

import numpy as np

from oracle import plogp_oracle as po

TIME_RTOL = 1e-12
TIE_MARGIN = 1e-9
SEG_IDS = po.SEGMENTED_IDS


def oracle_tables(w):
    return [po.Table(w.table_sizes(t), w.gaps[t], w.latency[t]) for t in range(w.n_tables)]


def oracle_sgrid(w):
    return po.SGrid(w.s_list) if w.s_list is not None else po.SGrid(lo=w.s_lo, hi=w.s_hi, step=w.s_step)


def _rel(a, b):
    return np.abs(a - b) / np.maximum(np.abs(b), 1e-300)


def _sub(t, ti, p_idx, m_idx):
    """[planes][P][m] slice of a device tensor for table ti as numpy."""
    import torch
    x = t[ti]
    dev = x.device
    x = x.index_select(1, torch.as_tensor(p_idx, device=dev)).index_select(2, torch.as_tensor(m_idx, device=dev))
    return x.cpu().numpy()


def _n_cand(w, m):
    if w.s_list is not None:
        return int(np.searchsorted(w.s_list, m, side="right"))
    top = min(int(m), w.s_hi)
    return (top - w.s_lo) // w.s_step + 1 if top >= w.s_lo else 0


def _valid_s(w, m, s):
    if _n_cand(w, m) == 0:
        return s == m
    if s > m or s <= 0:
        return False
    if w.s_list is not None:
        i = int(np.searchsorted(w.s_list, s))
        return i < len(w.s_list) and int(w.s_list[i]) == s
    return w.s_lo <= s <= w.s_hi and (s - w.s_lo) % w.s_step == 0


def _check_seg(w, t, sid, P, m, g_s, g_time, o_s, o_time, o_ru, where):
    """One segmented cell under the acceptance rule. Returns the oracle time for the GPU's pick."""
    if g_s == o_s:
        assert _rel(g_time, o_time) <= TIME_RTOL, (where, g_time, o_time)
        return o_time
    margin = (o_ru - o_time) / o_time
    assert margin <= TIE_MARGIN, "%s: segment size %d != oracle %d with margin %.3g" % (where, g_s, o_s, margin)
    assert _valid_s(w, m, g_s), "%s: %d is not a candidate segment size" % (where, g_s)
    alt = po.model(t, sid, P, m, g_s, w.k_mode)
    assert (alt - o_time) / o_time <= TIE_MARGIN, (where, alt, o_time)
    assert _rel(g_time, alt) <= TIME_RTOL, (where, g_time, alt)
    return alt


def check_prediction(w, ot, pred, tables=None, p_idx=None, m_idx=None) -> int:
    """Compare plogp_predict outputs with the oracle on the given tables / P indices / m indices."""
    tables = range(w.n_tables) if tables is None else tables
    p_idx = np.arange(w.n_P) if p_idx is None else np.asarray(p_idx)
    m_idx = np.arange(w.n_m) if m_idx is None else np.asarray(m_idx)
    Ps, ms = w.P_values()[p_idx], w.m[m_idx]
    sg = oracle_sgrid(w)
    n = 0
    for ti in tables:
        o = po.predict_grid(ot[ti], w.strategy_mask, Ps, ms, sg, w.k_mode)
        g_time = _sub(pred.time, ti, p_idx, m_idx)
        g_best = None if pred.best_s is None else _sub(pred.best_s, ti, p_idx, m_idx).view(np.uint32)
        for sid in range(po.N_STRATEGIES):
            if not (w.strategy_mask >> sid) & 1:
                assert np.isnan(g_time[sid]).all(), "disabled plane %d was written" % sid
                continue
            if sid in SEG_IDS and g_best is not None:
                q = SEG_IDS.index(sid)
                same = g_best[q] == o.best_s[q]
                assert (_rel(g_time[sid][same], o.time[sid][same]) <= TIME_RTOL).all(), (ti, sid)
                for ip, im in zip(*np.nonzero(~same)):
                    _check_seg(w, ot[ti], sid, int(Ps[ip]), int(ms[im]), int(g_best[q, ip, im]),
                               g_time[sid, ip, im], int(o.best_s[q, ip, im]), o.time[sid, ip, im],
                               o.seg_runner_up[q, ip, im], "table %d id %d P %d m %d" % (ti, sid, Ps[ip], ms[im]))
            else:
                r = _rel(g_time[sid], o.time[sid])
                assert (r <= TIME_RTOL).all(), "table %d id %d: max rel err %.3g" % (ti, sid, r.max())
            n += g_time[sid].size
    return n


def check_decision(w, ot, dec, tables=None, p_idx=None, m_idx=None) -> int:
    """Compare plogp_select_best outputs with the oracle's decision table."""
    tables = range(w.n_tables) if tables is None else tables
    p_idx = np.arange(w.n_P) if p_idx is None else np.asarray(p_idx)
    m_idx = np.arange(w.n_m) if m_idx is None else np.asarray(m_idx)
    Ps, ms = w.P_values()[p_idx], w.m[m_idx]
    sg = oracle_sgrid(w)
    mask = w.strategy_mask
    n = 0
    for ti in tables:
        o = po.predict_grid(ot[ti], mask, Ps, ms, sg, w.k_mode)
        od = po.select_grid(mask, o)
        g_id = _sub(dec.strategy, ti, p_idx, m_idx)
        g_s = _sub(dec.s_bytes, ti, p_idx, m_idx).view(np.uint32)
        g_t = _sub(dec.time, ti, p_idx, m_idx)
        for c, bits in ((0, mask & 0x3FF), (1, mask & 0x1C00)):
            if not bits:
                assert (g_id[c] == 255).all() and np.isnan(g_t[c]).all(), "collective %d has no strategy yet was written" % c
                continue
            same = (g_id[c] == od.strategy[c]) & (g_s[c] == od.s[c])
            assert (_rel(g_t[c][same], od.time[c][same]) <= TIME_RTOL).all(), (ti, c)
            for ip, im in zip(*np.nonzero(~same)):
                P, m = int(Ps[ip]), int(ms[im])
                gid, gs, gt = int(g_id[c, ip, im]), int(g_s[c, ip, im]), g_t[c, ip, im]
                where = "table %d coll %d P %d m %d" % (ti, c, P, m)
                assert (mask >> gid) & 1 and (gid < 10) == (c == 0), "%s: strategy %d not eligible" % (where, gid)
                best = od.time[c, ip, im]
                if gid in SEG_IDS:
                    q = SEG_IDS.index(gid)
                    alt = _check_seg(w, ot[ti], gid, P, m, gs, gt, int(o.best_s[q, ip, im]), o.time[gid, ip, im],
                                     o.seg_runner_up[q, ip, im], where)
                else:
                    assert gs == 0, where
                    alt = o.time[gid, ip, im]
                    assert _rel(gt, alt) <= TIME_RTOL, (where, gt, alt)
                if gid != int(od.strategy[c, ip, im]):
                    margin = (od.runner_up[c, ip, im] - best) / best
                    assert margin <= TIE_MARGIN, "%s: strategy %d != oracle %d with margin %.3g" % (
                        where, gid, od.strategy[c, ip, im], margin)
                assert (alt - best) / best <= TIE_MARGIN, (where, alt, best)
            n += g_id[c].size
    return n


def check_decision_cells(w, dec, t_idx, p_idx, m_idx, table_cache=None) -> int:
    """Decision cells given one by one (table, P index, m index), each re-decided by the oracle on its
    own (po.decide: every enabled strategy, exhaustive segment search) — for launch shapes whose whole
    tables the oracle cannot redo.  Both collectives of every sampled cell are checked."""
    import torch
    t_idx, p_idx, m_idx = (np.asarray(x, dtype=np.int64) for x in (t_idx, p_idx, m_idx))
    dev = dec.strategy.device
    ti, pi, mi = (torch.as_tensor(x, device=dev) for x in (t_idx, p_idx, m_idx))
    g_id = dec.strategy[ti, :, pi, mi].cpu().numpy()
    g_s = dec.s_bytes[ti, :, pi, mi].cpu().numpy().view(np.uint32)
    g_t = dec.time[ti, :, pi, mi].cpu().numpy()
    sg = oracle_sgrid(w)
    mask = w.strategy_mask
    Ps = w.P_values()
    cache = {} if table_cache is None else table_cache
    n = 0
    for i in range(len(t_idx)):
        t = int(t_idx[i])
        if t not in cache:
            cache[t] = po.Table(w.table_sizes(t), w.gaps[t], w.latency[t])
        tab = cache[t]
        P, m = int(Ps[p_idx[i]]), int(w.m[m_idx[i]])
        for c, bits in ((0, mask & 0x3FF), (1, mask & 0x1C00)):
            if not bits:
                continue
            sid, s, best, _ = po.decide(tab, c, mask, P, m, sg, w.k_mode)
            gid, gs, gt = int(g_id[i, c]), int(g_s[i, c]), float(g_t[i, c])
            where = "table %d coll %d P %d m %d" % (t, c, P, m)
            n += 1
            if gid == sid and gs == s:
                assert _rel(gt, best) <= TIME_RTOL, (where, gt, best)
                continue
            # another pick: only inside the tie margin, and with the oracle's time for that very pick
            assert (mask >> gid) & 1 and (gid < 10) == (c == 0), "%s: strategy %d not eligible" % (where, gid)
            if gid in SEG_IDS:
                assert _valid_s(w, m, gs), "%s: %d is not a candidate segment size" % (where, gs)
                alt = po.model(tab, gid, P, m, gs, w.k_mode)
            else:
                assert gs == 0, where
                alt = po.model(tab, gid, P, m, 0, w.k_mode)
            assert (alt - best) / best <= TIE_MARGIN, "%s: picked (%d, %d) at %.17g, oracle (%d, %d) at %.17g" % (
                where, gid, gs, alt, sid, s, best)
            assert _rel(gt, alt) <= TIME_RTOL, (where, gt, alt)
    return n
