// Greedy marginal-utility policy (host code): which stored form every KV cache entry gets on a
// storage tier of limited capacity.
//
// The paper's Design section defines Utility(i) = Freq(i) * (alpha * Quality(i, M_i, R_i) -
// size(i, M_i, R_i) / Bandwidth), states the problem as a multiple-choice knapsack and solves it
// greedily: among all entries take the move (compress further, or evict) whose marginal utility
// drop (Utility(i, m) - Utility(i, n)) / (size(i) * (m - n)), the utility lost per byte saved, is
// smallest, until everything left fits.  As in the textbook method it cites, only the
// LP-undominated options of an entry (the upper convex hull of its (size, utility) points together
// with eviction at (0, 0)) are walked, which makes the result optimal for the linear relaxation.
// size() is what kvh_level_bytes / kvh_plan_chunks report for the entry's stored form.
#include <stdint.h>

#include <algorithm>
#include <queue>
#include <vector>

#include "kvh.h"

namespace {

struct Point { uint64_t size; double util; int32_t option; };

// Is a/b < c/d for positive b, d?  Cross-multiplied in extended precision.
bool ratio_less(double a, uint64_t b, double c, uint64_t d)
{
    return (long double)a * (long double)d < (long double)c * (long double)b;
}

// The chain the greedy walks for one entry: its best point, then hull vertices of strictly smaller
// size, ending with eviction.
std::vector<Point> hull_of_entry(std::vector<Point> pts)
{
    pts.push_back(Point{0, 0.0, -1});
    Point best = pts[0];
    for (const Point &p : pts)
        if (p.util > best.util || (p.util == best.util && p.size < best.size)) best = p;
    std::vector<Point> lower;                            // smaller than best; per size the highest utility
    std::sort(pts.begin(), pts.end(), [](const Point &x, const Point &y) {
        return x.size != y.size ? x.size < y.size : (x.util != y.util ? x.util > y.util : x.option < y.option);
    });
    for (const Point &p : pts)
        if (p.size < best.size && (lower.empty() || lower.back().size != p.size)) lower.push_back(p);
    std::vector<Point> chain{best};
    Point cur = best;
    while (cur.size > 0) {
        const Point *next = nullptr;
        for (const Point &p : lower) {                   // ascending size: on equal slopes the smallest wins
            if (p.size >= cur.size) break;
            if (!next || ratio_less(cur.util - p.util, cur.size - p.size, cur.util - next->util, cur.size - next->size))
                next = &p;
        }
        chain.push_back(*next);
        cur = *next;
    }
    return chain;
}

struct Move { double drop; uint64_t saved; int32_t entry; };
struct MoveWorse {                                       // priority queue: smallest drop per byte first, then lowest entry
    bool operator()(const Move &x, const Move &y) const
    {
        if (ratio_less(y.drop, y.saved, x.drop, x.saved)) return true;
        if (ratio_less(x.drop, x.saved, y.drop, y.saved)) return false;
        return x.entry > y.entry;
    }
};

kvh_status assign(const double *freq, const kvh_option *options, const int32_t *option_begin, int n,
                  const kvh_tier *tier, const std::vector<int32_t> &cand, int32_t *choice, uint64_t *used_out,
                  double *utility_out)
{
    if (!(tier->bandwidth > 0.0)) return KVH_ERR_INVALID_ARG;
    std::vector<std::vector<Point>> chains(n);
    std::vector<int32_t> pos(n, 0);
    uint64_t used = 0;
    for (int32_t i : cand) {
        if (option_begin[i + 1] < option_begin[i]) return KVH_ERR_INVALID_ARG;
        std::vector<Point> pts;
        for (int32_t k = option_begin[i]; k < option_begin[i + 1]; ++k)
            pts.push_back(Point{options[k].size,
                                freq[i] * (tier->alpha * options[k].quality - (double)options[k].size / tier->bandwidth),
                                k - option_begin[i]});
        chains[i] = hull_of_entry(pts);
        used += chains[i][0].size;
    }
    std::priority_queue<Move, std::vector<Move>, MoveWorse> moves;
    auto push_next = [&](int32_t i) {
        const std::vector<Point> &ch = chains[i];
        const int32_t p = pos[i];
        if (p + 1 < (int32_t)ch.size())
            moves.push(Move{ch[p].util - ch[p + 1].util, ch[p].size - ch[p + 1].size, i});
    };
    for (int32_t i : cand) push_next(i);
    while (used > tier->capacity && !moves.empty()) {
        const Move m = moves.top();
        moves.pop();
        used -= m.saved;
        ++pos[m.entry];
        push_next(m.entry);
    }
    double total = 0.0;
    for (int32_t i : cand) {
        choice[i] = chains[i][pos[i]].option;
        total += chains[i][pos[i]].util;
    }
    if (used_out) *used_out = used;
    if (utility_out) *utility_out = total;
    return KVH_OK;
}

}  // namespace

extern "C" kvh_status kvh_policy_assign(const double *freq, const kvh_option *options, const int32_t *option_begin,
                                        int n_entries, const kvh_tier *tier, int32_t *choice_out,
                                        uint64_t *used_bytes, double *total_utility)
{
    if (!freq || !options || !option_begin || !tier || !choice_out || n_entries < 0) return KVH_ERR_INVALID_ARG;
    std::vector<int32_t> cand(n_entries);
    for (int i = 0; i < n_entries; ++i) cand[i] = i;
    return assign(freq, options, option_begin, n_entries, tier, cand, choice_out, used_bytes, total_utility);
}

extern "C" kvh_status kvh_policy_assign_tiers(const double *freq, const kvh_option *options,
                                              const int32_t *option_begin, int n_entries, const kvh_tier *tiers,
                                              int n_tiers, int32_t *tier_out, int32_t *choice_out)
{
    if (!freq || !options || !option_begin || !tiers || !tier_out || !choice_out || n_entries < 0 || n_tiers < 1)
        return KVH_ERR_INVALID_ARG;
    std::vector<int32_t> left(n_entries), choice(n_entries);
    for (int i = 0; i < n_entries; ++i) { left[i] = i; tier_out[i] = -1; choice_out[i] = -1; }
    for (int t = 0; t < n_tiers; ++t) {
        const kvh_status s = assign(freq, options, option_begin, n_entries, &tiers[t], left, choice.data(), nullptr,
                                    nullptr);
        if (s != KVH_OK) return s;
        std::vector<int32_t> next;
        for (int32_t i : left) {
            if (choice[i] >= 0) { tier_out[i] = t; choice_out[i] = choice[i]; }
            else next.push_back(i);
        }
        left.swap(next);
    }
    return KVH_OK;
}

// ---- a debugging aid for callers of the decode entry points -----------------------------------

// Two tokens mapped to the same page slot would make a load depend on the order in which tiles
// happen to run.  The kernels cannot see that; the caller can check its table on the host.
extern "C" kvh_status kvh_check_page_table(const int32_t *page_table, int64_t len, int32_t num_pages,
                                           int64_t *first_bad)
{
    if (!page_table || len < 0 || num_pages <= 0) return KVH_ERR_INVALID_ARG;
    std::vector<std::pair<int32_t, int64_t>> ids((size_t)len);
    for (int64_t i = 0; i < len; ++i) {
        if (page_table[i] < 0 || page_table[i] >= num_pages) {
            if (first_bad) *first_bad = i;
            return KVH_ERR_PAGE_OOB;
        }
        ids[(size_t)i] = {page_table[i], i};
    }
    std::sort(ids.begin(), ids.end());
    int64_t bad = -1;
    for (size_t i = 1; i < ids.size(); ++i)
        if (ids[i].first == ids[i - 1].first && (bad < 0 || ids[i].second < bad)) bad = ids[i].second;
    if (bad >= 0) {
        if (first_bad) *first_bad = bad;
        return KVH_ERR_INVALID_ARG;
    }
    return KVH_OK;
}
