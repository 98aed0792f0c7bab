"""Do the pins bite?  Each case plants one plausible mistake in the CPU checker (a dropped term, a wrong
sign or index, a swapped operand, an off-by-one) and runs the checker's own pin tests against the altered
checker: at least one pin has to fail.  The mistakes live here, in replacement functions that are patched
over the checker's for the length of one case; nothing outside the checker is touched."""
import itertools
import math

import numpy as np
import pytest

from oracle import spindlekv_oracle as O

import test_oracle_codebook
import test_oracle_compose
import test_oracle_decode
import test_oracle_evict
import test_oracle_plan


def _pins(module):
    """Every ``test_*`` function of a pin module as zero-argument callables (parametrised ones expanded)."""
    out = []
    for name in sorted(vars(module)):
        fn = getattr(module, name)
        if not (name.startswith("test_") and callable(fn)):
            continue
        marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
        if not marks:
            out.append((name, fn))
            continue
        axes = []
        for m in marks:
            names = [s.strip() for s in m.args[0].split(",")]
            rows = [v if len(names) > 1 else (v,) for v in m.args[1]]
            axes.append([dict(zip(names, row)) for row in rows])
        for combo in itertools.product(*axes):
            kw = {}
            for part in combo:
                kw.update(part)
            out.append((f"{name}[{sorted(kw)}]", lambda fn=fn, kw=kw: fn(**kw)))
    return out


def _failing_pins(modules):
    failed = []
    for module in modules:
        for name, call in _pins(module):
            try:
                call()
            except Exception:  # an assertion, or an error the mistake provokes (a shape, a division)
                failed.append(name)
    return failed


# ---- the planted mistakes ------------------------------------------------------------------------

def _attention(scale=True, mask="<=", axis=1, start_shift=0):
    def window_attention(q_win, k):
        q_win = np.asarray(q_win, dtype=np.float64)
        k = np.asarray(k, dtype=np.float64)
        w, d = q_win.shape
        l = k.shape[0]
        s = q_win @ k.T
        if scale:
            s = s / math.sqrt(d)
        pos_b = (l - w + start_shift) + np.arange(w)[:, None]
        cols = np.arange(l)[None, :]
        allowed = cols <= pos_b if mask == "<=" else cols < pos_b
        s = np.where(allowed, s, -np.inf)
        s = s - s.max(axis=axis, keepdims=True)
        e = np.exp(s)
        return e / e.sum(axis=axis, keepdims=True)
    return window_attention


def _accumulated(kind):
    def accumulated_scores(q_win, k, divide_by_distance=True):
        A = O.window_attention(q_win, k)
        l = k.shape[0]
        ac = A.sum(axis=0)
        if divide_by_distance:
            a = np.arange(l, dtype=np.float64)
            ac = ac / {"from_start": a + 1.0, "one_short": l - a + 1.0, "squared": (l - a) ** 2}[kind]
        return ac
    return accumulated_scores


def _group(kind):
    def group_scores(q_win_heads, k_heads, divide_by_distance=True):
        H_q, H_kv = q_win_heads.shape[0], k_heads.shape[0]
        h_n = H_q // H_kv
        out = np.zeros((H_kv, k_heads.shape[1]), dtype=np.float64)
        for j in range(H_kv):
            for g in range(h_n):
                i = j + H_kv * g if kind == "interleaved" else h_n * j + g
                out[j] += O.accumulated_scores(q_win_heads[i], k_heads[j], divide_by_distance)
            if kind != "sum":
                out[j] /= float(h_n)
        return out
    return group_scores


def _topk(kind):
    def arg_topk(scores, k):
        scores = np.asarray(scores, dtype=np.float64)
        idx = np.arange(scores.shape[0])
        if kind == "ties_high":
            order = np.lexsort((-idx, -scores))
        elif kind == "smallest":
            order = np.lexsort((idx, scores))
        else:  # unsorted output
            return np.lexsort((idx, -scores))[:k].astype(np.int32)
        return np.sort(order[:k]).astype(np.int32)
    return arg_topk


def _evict_window_dropped(q_win_heads, k_heads, k_ctx, divide_by_distance=True):
    w = q_win_heads.shape[1]
    H_kv, l, _ = k_heads.shape
    sc = O.group_scores(q_win_heads, k_heads, divide_by_distance)   # the window competes with the context
    keep = np.empty((H_kv, k_ctx + w), dtype=np.int32)
    for j in range(H_kv):
        keep[j] = O.arg_topk(sc[j], k_ctx + w)
    return {"keep": keep, "scores": sc[:, :l - w]}


def _magnitudes(kind):
    def magnitudes(gamma):
        gamma = np.asarray(gamma, dtype=np.float64)
        if kind == "l1":
            return np.abs(gamma).sum(axis=1)
        return (gamma * gamma).sum(axis=1)   # the square root forgotten
    return magnitudes


def _adjacency(kind):
    def adjacency(S, theta):
        if kind == "not_strict":
            up = np.triu(S >= theta, k=1)
        elif kind == "absolute":
            up = np.triu(np.abs(S) > theta, k=1)
        else:
            up = np.triu(S > theta, k=1)
        G = up | up.T
        np.fill_diagonal(G, True)
        return G
    return adjacency


def _greedy(kind):
    def codebook_greedy(G):
        G = np.asarray(G, dtype=bool)
        n = G.shape[0]
        live = np.ones(n, dtype=bool)
        s = G.sum(axis=1).astype(np.int64)
        ref = -np.ones(n, dtype=np.int32)
        centres, degs = [], []
        n_live = n
        while n_live > 0:
            masked = np.where(live, s, -1)
            if kind == "last_max":
                iota = int(n - 1 - np.argmax(masked[::-1]))
            elif kind == "min_degree":
                iota = int(np.argmin(np.where(live, s, n + 1)))
            else:
                iota = int(np.argmax(masked))
            eta = np.flatnonzero(G[iota] & live)
            ref[eta] = len(centres)
            centres.append(iota)
            degs.append(int(s[iota]))
            live[eta] = False
            n_live -= eta.shape[0]
            if kind != "static_degrees":
                s -= G[eta].sum(axis=0)
        return np.array(centres, dtype=np.int32), ref, np.array(degs, dtype=np.int64)
    return codebook_greedy


def _endpoints_swapped(r_c, beta):
    alpha = 0.5 * (1.0 + beta)
    if beta < r_c <= alpha:
        return beta, 2.0 * r_c - beta
    if alpha < r_c <= 1.0:
        return 2.0 * r_c - 1.0, 1.0
    raise O.BudgetError("outside")


def _endpoints_alpha_is_half(r_c, beta):
    if beta < r_c <= 0.5:
        return 2.0 * r_c - beta, beta
    if 0.5 < r_c <= 1.0:
        return 1.0, 2.0 * r_c - 1.0
    raise O.BudgetError("outside")


def _layer_ratio_over_m(r_first, r_last, m, lam, r_c):
    return r_c if m == 1 else r_first + (r_last - r_first) / float(m) * float(lam)


def _ratio_over_whole_length(reserved_tokens, l, l_w):
    if l - l_w <= 0:
        raise O.BudgetError("short")
    return (float(reserved_tokens) - float(l_w)) / float(l)


def _reconstruct_centre_magnitude(C, ref, mag):
    C = np.asarray(C, dtype=np.float64)
    mag = np.asarray(mag, dtype=np.float64)
    # every token takes the magnitude of the first token that shares its entry, instead of its own
    first = {}
    for t, r in enumerate(ref):
        first.setdefault(int(r), t)
    return C[ref] * np.array([mag[first[int(r)]] for r in ref])[:, None]


def _match(kind):
    def match_entries(C, gamma_new, theta):
        C = np.asarray(C, dtype=np.float64)
        g = O.normalise(gamma_new, O.magnitudes(gamma_new))
        S = g @ O.normalise(C, O.magnitudes(C)).T if C.shape[0] else np.zeros((g.shape[0], 0))
        ref = -np.ones(g.shape[0], dtype=np.int32)
        for t in range(g.shape[0]):
            if S.shape[1] and S[t].max() > theta:
                if kind == "first_suitable":
                    ref[t] = int(np.flatnonzero(S[t] > theta)[0])
                else:   # the last of equal maxima
                    ref[t] = int(S.shape[1] - 1 - np.argmax(S[t][::-1]))
        return ref, S
    return match_entries


def _normalise_by_square(gamma, m):
    gamma = np.asarray(gamma, dtype=np.float64)
    safe = np.where(m > 0.0, m * m, 1.0)
    return np.where(m[:, None] > 0.0, gamma / safe[:, None], 0.0)


def _plan_with(rounding):
    def plan_layers(n_layers, n_shallow, seq_lens, l_w, beta, reserve_ratio=None, budget_tokens=None):
        B = len(seq_lens)
        if n_shallow == -1:
            if rounding == "literal_keeps_a_split":
                return _ORIGINAL["plan_layers"](n_layers, n_layers // 2, seq_lens, l_w, beta, reserve_ratio, budget_tokens)
            mode, ratio, k_ctx = plan_layers(n_layers, 0, seq_lens, l_w, beta, reserve_ratio, budget_tokens)
            return np.full(n_layers, O.MODE_EVICT | O.MODE_CODEBOOK, dtype=np.int32), ratio, k_ctx
        m_deep = n_layers - n_shallow
        mode = np.array([O.MODE_CODEBOOK if lam < n_shallow else O.MODE_EVICT for lam in range(n_layers)], dtype=np.int32)
        ratio = np.ones((n_layers, B), dtype=np.float64)
        k_ctx = np.zeros((n_layers, B), dtype=np.int32)
        for s, l in enumerate(seq_lens):
            l_c = l - l_w
            if l_c <= 0:
                raise O.BudgetError("short")
            k_ctx[:n_shallow, s] = l_c
            if m_deep == 0:
                continue
            rl = float(budget_tokens) if budget_tokens is not None else float(reserve_ratio) * float(l)
            r_c = O.context_reserve_ratio(rl, l, l_w)
            r0, r1 = O.pyramid_endpoints(r_c, beta)
            for lam in range(m_deep):
                r = O.layer_ratio(r0, r1, m_deep, lam, r_c)
                ratio[n_shallow + lam, s] = r
                k = math.ceil(r * float(l_c)) if rounding == "ceil" else math.floor(r * float(l))
                k_ctx[n_shallow + lam, s] = min(l_c, int(k))
        return mode, ratio, k_ctx
    return plan_layers


def _shallow(kind):
    def codebook_shallow(gamma, theta, G_override=None):
        gamma = np.asarray(gamma, dtype=np.float64)
        mag = O.magnitudes(gamma)
        ghat = O.normalise(gamma, mag)
        S = ghat @ ghat.T
        G = O.adjacency(S, theta) if G_override is None else np.asarray(G_override, dtype=bool)
        centres, ref, degs = O.codebook_greedy(G)
        C = gamma[centres] if kind == "raw_centres" else ghat[centres]
        if kind == "mean_of_members":
            C = np.stack([ghat[ref == e].mean(axis=0) for e in range(len(centres))])
        return {"mag": mag, "ref": ref, "centres": centres, "C": C, "S": S, "G": G, "pick_degree": degs}
    return codebook_shallow


def _layer(kind):
    def spindle_layer(q_win_heads, k_heads, v_heads, k_ctx, theta_k, theta_v):
        ev = O.evict_deep(q_win_heads, k_heads, k_ctx)
        cb_k, cb_v = [], []
        for j in range(k_heads.shape[0]):
            rows = np.arange(k_heads.shape[1]) if kind == "all_tokens" else ev["keep"][j]
            tk, tv = (theta_v, theta_k) if kind == "thresholds_swapped" else (theta_k, theta_v)
            cb_k.append(O.codebook_shallow(O.gather_rows(k_heads[j], rows), tk))
            cb_v.append(O.codebook_shallow(O.gather_rows(v_heads[j], rows), tv))
        return {"keep": ev["keep"], "scores": ev["scores"], "cb_k": cb_k, "cb_v": cb_v}
    return spindle_layer


def _repeat_heads_interleaved(q_win_heads, k_heads, v_heads, k_ctx, theta_k, theta_v):
    H_q, w = q_win_heads.shape[0], q_win_heads.shape[1]
    H_kv, l, _ = k_heads.shape
    h_n = H_q // H_kv
    keep = np.empty((H_q, k_ctx + w), dtype=np.int32)
    scores = np.empty((H_q, l - w), dtype=np.float64)
    for i in range(H_q):
        ev = O.evict_deep(q_win_heads[i:i + 1], k_heads[i % H_kv:i % H_kv + 1], k_ctx)
        keep[i], scores[i] = ev["keep"][0], ev["scores"][0]
    union = keep.reshape(H_kv, h_n * (k_ctx + w))
    cb_k = [O.codebook_shallow(O.gather_rows(k_heads[j], union[j]), theta_k) for j in range(H_kv)]
    cb_v = [O.codebook_shallow(O.gather_rows(v_heads[j], union[j]), theta_v) for j in range(H_kv)]
    return {"keep": keep, "scores": scores, "union": union, "cb_k": cb_k, "cb_v": cb_v}


def _ratio_entries_over_all_tokens(l, kept, entries_k, entries_v):
    h = len(entries_k)
    return (2.0 * h * kept) / (2.0 * h * l), (float(sum(entries_k)) + float(sum(entries_v))) / (2.0 * h * l)


def _extend_without_offset(C, gamma_new, theta, ref_override=None, G_override=None):
    out = _ORIGINAL["codebook_extend"](C, gamma_new, theta, ref_override, G_override)
    if out["left"].size:
        out["ref"][out["left"]] -= np.asarray(C).shape[0]
    return out


def _rope(kind):
    def rope(x, positions, base=10000.0):
        x = np.asarray(x, dtype=np.float64)
        d = x.shape[-1]
        h = d // 2
        ang = np.asarray(positions, dtype=np.float64)[..., None] * O.rope_frequencies(d, base)
        c, s_ = np.cos(ang), np.sin(ang)
        if kind == "clockwise":
            s_ = -s_
        if kind == "neighbouring_pairs":               # (2i, 2i+1) instead of (i, i + d/2)
            a, b = x[..., 0::2], x[..., 1::2]
            out = np.empty_like(x)
            out[..., 0::2], out[..., 1::2] = a * c - b * s_, b * c + a * s_
            return out
        a, b = x[..., :h], x[..., h:]
        return np.concatenate([a * c - b * s_, b * c + a * s_], axis=-1)
    return rope


def _frequencies_of_half_the_dimension(d, base=10000.0):
    return np.asarray(base, dtype=np.float64) ** (-1.0 * np.arange(d // 2, dtype=np.float64) / float(d))


def _decode(kind):
    def decode_attention(q, pos_q, C_K, r_K, m_K, C_V, r_V, m_V, positions=None, base=10000.0):
        q = np.asarray(q, dtype=np.float64)
        n, d = np.asarray(r_K).shape[0], q.shape[1]
        positions = np.arange(n) if (positions is None or kind == "positions_ignored") else np.asarray(positions)
        K = O.reconstruct(C_K, r_K, np.ones(n) if kind == "key_magnitude_dropped" else m_K)
        K = K if kind == "keys_not_rotated" else O.rope(K, positions, base)
        V = O.reconstruct(C_V, r_V, np.ones(n) if kind == "value_magnitude_dropped" else m_V)
        qr = q if kind == "query_not_rotated" else O.rope(q, np.full(q.shape[0], pos_q), base)
        s = (qr @ K.T) / (1.0 if kind == "no_scale" else math.sqrt(d))
        s = s - s.max(axis=1, keepdims=True)
        e = np.exp(s)
        A = e / e.sum(axis=1, keepdims=True)
        return {"out": A @ V, "A": A}
    return decode_attention


_ORIGINAL = {"plan_layers": O.plan_layers, "codebook_extend": O.codebook_extend}

_EVICT = (test_oracle_evict, test_oracle_compose)
_CODEBOOK = (test_oracle_codebook, test_oracle_compose)
_PLAN = (test_oracle_plan, test_oracle_compose)
_DECODE = (test_oracle_decode,)

MUTANTS = [
    ("logits not scaled by 1/sqrt(d)", "window_attention", _attention(scale=False), _EVICT),
    ("a query does not see its own position", "window_attention", _attention(mask="<"), _EVICT),
    ("softmax over the queries instead of the keys", "window_attention", _attention(axis=0), _EVICT),
    ("window placed one position early", "window_attention", _attention(start_shift=-1), _EVICT),
    ("distance counted from the start", "accumulated_scores", _accumulated("from_start"), _EVICT),
    ("distance one too large", "accumulated_scores", _accumulated("one_short"), _EVICT),
    ("distance squared", "accumulated_scores", _accumulated("squared"), _EVICT),
    ("query heads interleaved over the KV heads", "group_scores", _group("interleaved"), _EVICT),
    ("group sum instead of group mean", "group_scores", _group("sum"), _EVICT),
    ("ties go to the higher index", "arg_topk", _topk("ties_high"), _EVICT),
    ("the k smallest", "arg_topk", _topk("smallest"), _EVICT),
    ("kept positions not ascending", "arg_topk", _topk("unsorted"), _EVICT),
    ("window competes instead of being reserved", "evict_deep", _evict_window_dropped, _EVICT),
    ("L1 norm", "magnitudes", _magnitudes("l1"), _CODEBOOK),
    ("square root forgotten", "magnitudes", _magnitudes("no_sqrt"), _CODEBOOK),
    ("threshold not strict", "adjacency", _adjacency("not_strict"), _CODEBOOK),
    ("absolute cosine", "adjacency", _adjacency("absolute"), _CODEBOOK),
    ("last of equal degrees", "codebook_greedy", _greedy("last_max"), _CODEBOOK),
    ("smallest degree first", "codebook_greedy", _greedy("min_degree"), _CODEBOOK),
    ("degrees never updated", "codebook_greedy", _greedy("static_degrees"), _CODEBOOK),
    ("pyramid upside down", "pyramid_endpoints", _endpoints_swapped, _PLAN),
    ("alpha taken as 1/2", "pyramid_endpoints", _endpoints_alpha_is_half, _PLAN),
    ("interpolation over m instead of m-1", "layer_ratio", _layer_ratio_over_m, _PLAN),
    ("ratio over the whole length", "context_reserve_ratio", _ratio_over_whole_length, _PLAN),
    ("division by the squared norm", "normalise", _normalise_by_square, _CODEBOOK),
    ("k rounded up", "plan_layers", _plan_with("ceil"), _PLAN),
    ("k taken from the whole length", "plan_layers", _plan_with("whole_length"), _PLAN),
    ("literal composition keeps a shallow half", "plan_layers", _plan_with("literal_keeps_a_split"), _PLAN),
    ("CodeBook of raw centre rows", "codebook_shallow", _shallow("raw_centres"), _CODEBOOK),
    ("CodeBook of member means", "codebook_shallow", _shallow("mean_of_members"), _CODEBOOK),
    ("CodeBooks over all tokens instead of the kept ones", "spindle_layer", _layer("all_tokens"), _CODEBOOK),
    ("K and V thresholds swapped", "spindle_layer", _layer("thresholds_swapped"), _CODEBOOK),
    ("repeat variant maps query heads round-robin", "spindle_layer_repeat", _repeat_heads_interleaved, _CODEBOOK),
    ("r2 over all tokens", "reserve_ratio_layer", _ratio_entries_over_all_tokens, _PLAN),
    ("appended entries keep their local numbers", "codebook_extend", _extend_without_offset, _CODEBOOK),
    ("reconstruction with a shared magnitude", "reconstruct", _reconstruct_centre_magnitude, _CODEBOOK),
    ("first suitable entry instead of the most similar", "match_entries", _match("first_suitable"), _CODEBOOK),
    ("last of equally similar entries", "match_entries", _match("last_max"), _CODEBOOK),
    ("rotation clockwise", "rope", _rope("clockwise"), _DECODE),
    ("rotation pairs neighbouring elements", "rope", _rope("neighbouring_pairs"), _DECODE),
    ("frequencies base**(-i/d)", "rope_frequencies", _frequencies_of_half_the_dimension, _DECODE),
    ("query not rotated", "decode_attention", _decode("query_not_rotated"), _DECODE),
    ("rebuilt keys not rotated", "decode_attention", _decode("keys_not_rotated"), _DECODE),
    ("cached tokens rotated at their list index", "decode_attention", _decode("positions_ignored"), _DECODE),
    ("key magnitudes dropped", "decode_attention", _decode("key_magnitude_dropped"), _DECODE),
    ("value magnitudes dropped", "decode_attention", _decode("value_magnitude_dropped"), _DECODE),
    ("decode scores not scaled by 1/sqrt(d)", "decode_attention", _decode("no_scale"), _DECODE),
]


def test_pins_pass_on_the_checker_as_it_stands():
    assert _failing_pins((test_oracle_evict, test_oracle_codebook, test_oracle_plan, test_oracle_compose,
                          test_oracle_decode)) == []


@pytest.mark.parametrize("what,attr,replacement,modules", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(monkeypatch, what, attr, replacement, modules):
    monkeypatch.setattr(O, attr, replacement)
    failed = _failing_pins(modules)
    assert failed, f"no pin notices: {what}"
