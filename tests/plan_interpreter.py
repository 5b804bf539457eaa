"""Executes a step plan (the int32 words pasta_step_begin uploads) with NumPy, unit by unit, the way
the kernels are meant to: every t-unit and w-unit yields partial (m, l, O) rows, the merge combines
them; the rows of a unit marked final go to the output as they are, and must then be the only rows of their
(query, head) pairs.  It lets the planner be checked against the oracle without a GPU.  Tests only."""
import numpy as np

# header word indices (pasta_plan.h)
(PH_MAGIC, PH_N_QUERIES, PH_N_APPEND, PH_N_TREQ, PH_N_TUNITS, PH_N_WUNITS, PH_T_ROWS, PH_ROWS, PH_T_GRID,
 PH_OFF_APPEND, PH_OFF_QUERY, PH_OFF_TREQ, PH_OFF_TRANGE, PH_OFF_TUNIT, PH_OFF_TCTA, PH_OFF_WUNIT, PH_OFF_PAGES,
 PH_OFF_PMETA, PH_OFF_VIS, PH_OFF_TQ, PH_OFF_APOS, PH_OFF_QPOS, PH_TOTAL_WORDS, PH_N_DUNITS, PH_OFF_DUNIT,
 PH_OFF_DRANGE, PH_N_PARTIAL) = range(27)
PQ, PT, PU, PW = 4, 6, 12, 4
TILE_PAGES, PAGE = 8, 16
STATS = {'flagged': 0, 'pages': 0}    # pages the plans marked as visible in full to every thread, of all pages walked


def run_plan(w, K, V, q, n_kv_heads):
    """w: plan words; K, V: [n_pages, 16, Hkv, d] float64; q: [n, Hq, d] float64 -> out [n, Hq, d], lse [n, Hq]."""
    assert w[PH_MAGIC] == 0x50415354 and w[PH_TOTAL_WORDS] == len(w)
    n, Hq, d = q.shape
    G = Hq // n_kv_heads
    scale = 1.0 / np.sqrt(d)
    rows = int(w[PH_ROWS]); t_rows = int(w[PH_T_ROWS])
    m = np.full(rows, np.nan); l = np.full(rows, np.nan); O = np.full((rows, d), np.nan)
    pages, pmeta = w[w[PH_OFF_PAGES]:], w[w[PH_OFF_PMETA]:]
    written = np.zeros(rows, dtype=int)

    # every t-unit belongs to exactly one CTA range, ranges are contiguous and cover all units
    cta = w[w[PH_OFF_TCTA]: w[PH_OFF_TCTA] + 2 * w[PH_T_GRID]].reshape(-1, 2)
    if w[PH_N_TUNITS]:
        assert cta[0, 0] == 0 and cta[-1, 1] == w[PH_N_TUNITS]
        assert np.all(cta[1:, 0] == cta[:-1, 1]) and np.all(cta[:, 1] > cta[:, 0])

    # assigned units, then the units the CTAs share out at run time (same record, a table of their own)
    recs = [w[w[PH_OFF_TUNIT] + u * PU: w[PH_OFF_TUNIT] + (u + 1) * PU] for u in range(w[PH_N_TUNITS])]
    recs += [w[w[PH_OFF_DUNIT] + u * PU: w[PH_OFF_DUNIT] + (u + 1) * PU] for u in range(w[PH_N_DUNITS])]
    STATS['dunits'] = STATS.get('dunits', 0) + int(w[PH_N_DUNITS])
    covered = {}
    final = set()                           # partial rows that are the whole result of their (query, head) pair
    STATS['final_units'] = STATS.get('final_units', 0) + sum(int(rec[11]) for rec in recs)
    # the header's count of units that leave partial rows (0 = the library does not launch the merge)
    assert w[PH_N_PARTIAL] == sum(1 - int(rec[11]) for rec in recs) + w[PH_N_WUNITS]
    STATS['no_merge_plans'] = STATS.get('no_merge_plans', 0) + int(w[PH_N_PARTIAL] == 0)
    for u, rec in enumerate(recs):
        treq, g, tb, te, row_base = rec[:5]
        T = w[PH_OFF_TREQ] + treq * PT
        page_off, n_pages, n_thr, n_str, vis_off, tq_off = w[T:T + PT]
        assert list(rec[5:11]) == [page_off, n_pages, n_thr, n_str, vis_off, tq_off]     # the unit repeats its t-request
        assert 0 <= tb < te <= -(-n_pages // TILE_PAGES)
        covered.setdefault((int(treq), int(g)), []).append((int(tb), int(te), -(-int(n_pages) // TILE_PAGES)))
        vis = w[w[PH_OFF_VIS] + vis_off: w[PH_OFF_VIS] + vis_off + n_thr * n_str].reshape(n_thr, n_str)
        tq = w[w[PH_OFF_TQ] + tq_off: w[PH_OFF_TQ] + tq_off + n_thr]
        for ti in range(n_thr):
            for hl in range(G):
                h = g * G + hl
                s_all, v_all = [], []
                for pi in range(tb * TILE_PAGES, min(te * TILE_PAGES, n_pages)):
                    page, meta = pages[page_off + pi], pmeta[page_off + pi]
                    thr = vis[ti, meta & 4095] - ((meta >> 12) & 0x3FFFF) * PAGE
                    cnt = int(np.clip(thr, 0, PAGE))
                    if meta & (1 << 30):        # the plan claims that no row needs a mask on this page
                        assert cnt == PAGE, (u, ti, pi)
                    STATS['flagged'], STATS['pages'] = STATS['flagged'] + bool(meta & (1 << 30)), STATS['pages'] + 1
                    s_all.append(K[page, :cnt, g] @ q[tq[ti], h] * scale)
                    v_all.append(V[page, :cnt, g])
                s = np.concatenate(s_all); v = np.concatenate(v_all)
                row = row_base + ti * G + hl
                written[row] += 1
                assert rec[11] in (0, 1)
                if rec[11]:
                    final.add(int(row))
                if len(s) == 0:
                    m[row], l[row], O[row] = -np.inf, 0.0, 0.0
                else:
                    m[row] = s.max(); e = np.exp(s - m[row]); l[row] = e.sum(); O[row] = e @ v

    for spans in covered.values():          # the units of a run tile it exactly: every tile once
        spans.sort()
        assert spans[0][0] == 0 and spans[-1][1] == spans[0][2]
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))

    for u in range(w[PH_N_WUNITS]):
        qi, g, page_off, n_tok = w[w[PH_OFF_WUNIT] + u * PW: w[PH_OFF_WUNIT] + (u + 1) * PW]
        assert n_tok > 0
        for hl in range(G):
            h = g * G + hl
            ks = np.concatenate([K[pages[page_off + k], :, g] for k in range(-(-n_tok // PAGE))])[:n_tok]
            vs = np.concatenate([V[pages[page_off + k], :, g] for k in range(-(-n_tok // PAGE))])[:n_tok]
            s = ks @ q[qi, h] * scale
            row = t_rows + u * G + hl
            written[row] += 1
            m[row] = s.max(); e = np.exp(s - m[row]); l[row] = e.sum(); O[row] = e @ vs
    assert np.all(written == 1), "every partial row is written exactly once"

    out = np.zeros((n, Hq, d)); lse = np.zeros((n, Hq))
    tr = w[w[PH_OFF_TRANGE]:]
    for i in range(n):
        treq, tidx, w0, nw = w[w[PH_OFF_QUERY] + i * PQ: w[PH_OFF_QUERY] + (i + 1) * PQ]
        for h in range(Hq):
            g, hl = divmod(h, G)
            rows_i = []
            if treq >= 0:
                for u in range(tr[(treq * n_kv_heads + g) * 2], tr[(treq * n_kv_heads + g) * 2 + 1]):
                    assert w[w[PH_OFF_TUNIT] + u * PU] == treq and w[w[PH_OFF_TUNIT] + u * PU + 1] == g
                    rows_i.append(w[w[PH_OFF_TUNIT] + u * PU + 4] + tidx * G + hl)
                dr = w[w[PH_OFF_DRANGE]:]
                for u in range(dr[(treq * n_kv_heads + g) * 2], dr[(treq * n_kv_heads + g) * 2 + 1]):
                    assert w[w[PH_OFF_DUNIT] + u * PU] == treq and w[w[PH_OFF_DUNIT] + u * PU + 1] == g
                    rows_i.append(w[w[PH_OFF_DUNIT] + u * PU + 4] + tidx * G + hl)
            rows_i += [t_rows + (w0 + g * nw + k) * G + hl for k in range(nw)]
            if any(int(r) in final for r in rows_i):      # written by the unit itself: nothing else may contribute
                assert len(rows_i) == 1
            elif len(rows_i) == 1 and nw == 0:            # a lone unit is final unless its request has w-units
                qt = w[w[PH_OFF_QUERY]: w[PH_OFF_QUERY] + n * PQ].reshape(n, PQ)
                assert np.any(qt[qt[:, 0] == treq, 3] > 0)
            rows_i = [r for r in rows_i if l[r] > 0]
            ms = max(m[r] for r in rows_i)
            L = sum(np.exp(m[r] - ms) * l[r] for r in rows_i)
            out[i, h] = sum(np.exp(m[r] - ms) * O[r] for r in rows_i) / L
            lse[i, h] = ms + np.log(L)
    return out, lse
