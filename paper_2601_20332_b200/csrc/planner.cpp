// Host planner: which positions are active, buffer, transient, far-field,
// computed and visible in the next step.  Integer logic only.
//
// Section 4.2 of the paper: the external window is a fixed-length prefix of
// the undecoded region and stays put within a phase; the internal window is
// the front of its still-undecoded part and slides right as tokens decode;
// buffer = external \ (active U decoded-in-phase); undecoded tokens outside
// the external window are pruned.  Section 4.3: a phase is one refresh step
// (everything visible is computed) followed by normal steps (active tokens and
// recently decoded tokens are computed).  Adaptive termination (Section 4.2): once an
// end-of-sequence token has been generated, undecoded positions after it are never activated
// again (they stay far-field) and the sequence is done when nothing undecoded precedes it.
// Staggered refresh (a variant for batches, which the paper does not discuss): sequence i of n shifts its
// phase clock by i * R / n steps, so that the batch's refresh steps do not all fall on the same step.
#include <algorithm>
#include <climits>

#include "wd_internal.h"

wd_status wd_plan_seq(const WdSeq& s, int32_t A, int32_t B, int32_t R, int32_t T, WdSeqPlan* out) {
    if (!out) return WD_ERR_NULL;
    if (A < 1 || B < 0 || R < 1 || T < 0) return WD_ERR_BAD_PARAM;
    WdSeqPlan& p = *out;
    p = WdSeqPlan();
    const int32_t S = (int32_t)s.ids.size();

    // first generated end-of-sequence token in position order (tokens that were given do not count)
    int32_t limit = S;
    if (s.eos_id >= 0)
        for (int32_t i = 0; i < S; ++i)
            if (s.decoded[i] && s.ids[i] == s.eos_id && s.dec_step[i] != INT32_MIN) { limit = i; break; }

    int32_t n_undecoded = 0;
    for (int32_t i = 0; i < limit; ++i) n_undecoded += s.decoded[i] ? 0 : 1;
    if (n_undecoded == 0) { p.done = true; return WD_OK; }

    // does the stored external window still hold an undecoded token (before the limit)?
    bool window_alive = false;
    for (int32_t i : s.wex) if (!s.decoded[i] && i < limit) { window_alive = true; break; }
    p.refresh = (s.t == 0) || (s.since >= R) || !window_alive;
    {
        // staggered refresh (variant): this sequence's second refresh comes `offset` steps after the first
        const int32_t offset = wd_stagger_offset(s.stagger_i, s.stagger_n, R);
        if (offset > 0 && offset < R && s.t == offset) p.refresh = true;
    }

    if (p.refresh) {
        // long arithmetic: A + B may exceed int32 for "window = everything" callers
        const int64_t want = std::min<int64_t>((int64_t)A + (int64_t)B, n_undecoded);
        p.wex.reserve((size_t)want);
        for (int32_t i = 0; i < limit && (int64_t)p.wex.size() < want; ++i)
            if (!s.decoded[i]) p.wex.push_back(i);
    } else {
        p.wex = s.wex;
    }

    // walk the external window once: undecoded members fill the internal
    // window first, the rest is buffer; decoded members were decoded in this
    // phase and are recomputed while young enough
    std::vector<uint8_t> live((size_t)S, 0);            // undecoded window members still in play
    for (int32_t i : p.wex) {
        if (!s.decoded[i]) {
            if (i >= limit) continue;                       // cut off by an end-of-sequence token
            live[i] = 1;
            if ((int32_t)p.active.size() < A) p.active.push_back(i);
            else p.buffer.push_back(i);
        } else {
            const int64_t age = (int64_t)s.t - (int64_t)s.dec_step[i];
            if (age >= 1 && age <= T) p.transient.push_back(i);
        }
    }

    // one pass over the sequence for the position-ordered lists
    for (int32_t i = 0; i < S; ++i) {
        if (s.decoded[i]) { p.decoded.push_back(i); p.vis.push_back(i); }
        else if (live[i]) p.vis.push_back(i);
        else p.far_field.push_back(i);
    }
    if (p.refresh && s.refresh_mode == WD_REFRESH_WINDOW && s.t > 0) {
        // variant (not in the paper): only the new window and the tokens decoded during the phase
        // that just ended are recomputed; s.phase_start is still that phase's first step
        for (int32_t i : p.vis)
            if (!s.decoded[i] || (s.dec_step[i] != INT32_MIN && s.dec_step[i] >= s.phase_start)) p.rows.push_back(i);
    } else if (p.refresh) {
        p.rows = p.vis;
    } else {
        p.rows.resize(p.active.size() + p.transient.size());
        std::merge(p.active.begin(), p.active.end(), p.transient.begin(), p.transient.end(),
                   p.rows.begin());
    }
    p.vis_contiguous = !p.vis.empty() && p.vis.back() == (int32_t)p.vis.size() - 1;
    return WD_OK;
}

void wd_commit_seq(WdSeq& s, const WdSeqPlan& plan, const int32_t* positions,
                   const int32_t* token_ids, int32_t n) {
    if (plan.done) return;
    if (plan.refresh) {
        s.wex = plan.wex;
        s.phase_start = s.t;
        s.since = 0;
    }
    for (int32_t i = 0; i < n; ++i) {
        const int32_t pos = positions[i];
        s.ids[pos] = token_ids[i];
        s.decoded[pos] = 1;
        s.dec_step[pos] = s.t;
    }
    s.t += 1;
    s.since += 1;
}

// ---- count-level shadow (see WdCount) ----------------------------------------------------

void wd_count_init(WdCount& c, const WdSeq& s) {
    c = WdCount();
    for (uint8_t d : s.decoded) (d ? c.decoded : c.undecoded) += 1;
    c.t = s.t;
    c.since = s.since;
    c.refresh_mode = s.refresh_mode;
    c.stagger_i = s.stagger_i;
    c.stagger_n = s.stagger_n;
    c.wex_size = (int32_t)s.wex.size();
    for (int32_t i : s.wex) c.w_alive += s.decoded[i] ? 0 : 1;
    // tokens unmasked at each step of the running phase, oldest first
    if (!s.wex.empty() && s.t > s.phase_start) {
        c.hist.assign((size_t)(s.t - s.phase_start), 0);
        for (int32_t i : s.wex)
            if (s.decoded[i] && s.dec_step[i] >= s.phase_start) c.hist[(size_t)(s.dec_step[i] - s.phase_start)] += 1;
    }
}

wd_status wd_count_plan(const WdCount& c, int32_t A, int32_t B, int32_t R, int32_t T, int32_t k, WdCountPlan* out) {
    if (!out) return WD_ERR_NULL;
    if (A < 1 || B < 0 || R < 1 || T < 0 || k < 0) return WD_ERR_BAD_PARAM;
    WdCountPlan& p = *out;
    p = WdCountPlan();
    if (c.undecoded == 0) { p.done = true; return WD_OK; }
    p.refresh = (c.t == 0) || (c.since >= R) || (c.w_alive == 0);
    {
        const int32_t offset = wd_stagger_offset(c.stagger_i, c.stagger_n, R);
        if (offset > 0 && offset < R && c.t == offset) p.refresh = true;
    }
    int32_t w_alive = c.w_alive;
    if (p.refresh) {
        p.n_wex = (int32_t)std::min<int64_t>((int64_t)A + (int64_t)B, c.undecoded);
        w_alive = p.n_wex;
    } else {
        p.n_wex = c.wex_size;
        // tokens unmasked at the last min(T, steps in this phase) steps are still recomputed
        const int32_t n_hist = (int32_t)c.hist.size();
        for (int32_t age = 1; age <= T && age <= n_hist; ++age) p.n_transient += c.hist[(size_t)(n_hist - age)];
    }
    p.n_active = std::min(A, w_alive);
    p.n_vis = c.decoded + w_alive;
    p.window_refresh = p.refresh && c.refresh_mode == WD_REFRESH_WINDOW && c.t > 0;
    p.prev_phase_start = c.t - c.since;
    int32_t prev_phase_tokens = 0;
    for (int32_t h : c.hist) prev_phase_tokens += h;
    p.n_rows = p.window_refresh ? p.n_wex + prev_phase_tokens : (p.refresh ? p.n_vis : p.n_active + p.n_transient);
    p.n_unmask = std::min(k, p.n_active);
    return WD_OK;
}

void wd_count_commit(WdCount& c, const WdCountPlan& p) {
    if (p.done) return;
    if (p.refresh) {
        c.wex_size = p.n_wex;
        c.w_alive = p.n_wex;
        c.since = 0;
        c.hist.clear();
    }
    c.undecoded -= p.n_unmask;
    c.decoded += p.n_unmask;
    c.w_alive -= p.n_unmask;
    c.hist.push_back(p.n_unmask);
    c.t += 1;
    c.since += 1;
}
