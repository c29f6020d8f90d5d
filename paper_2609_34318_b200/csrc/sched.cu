// The load-driven DCP scheduler (host only): closed-form targets and Algorithm 1 with the lazy heaps
// of Section 5.1.3. No device code lives here; the file is a .cu only so that one compiler builds the
// whole library.
//
// Exactness: every feasibility test and every comparison of per-rank loads is done on integers
// (loads are kept as sums of s^2, per-rank values are compared by cross-multiplication in 128 bits),
// so the heap search makes the very placements a scan of all open groups would make.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <queue>
#include <vector>

#include "../../include/hydra_attn.h"
#include "../../include/hydra_sched.h"

namespace {

using u128 = unsigned __int128;

inline bool is_pow2(int64_t x) { return x >= 1 && (x & (x - 1)) == 0; }
inline int log2i(int64_t x) { int j = 0; while ((int64_t{1} << j) < x) ++j; return j; }

// smallest power of two t with t * den >= num (num, den > 0)
inline int64_t ceil2_ratio(u128 num, u128 den)
{
    int64_t t = 1;
    while (static_cast<u128>(t) * den < num) t <<= 1;
    return t;
}

inline int32_t cp_degree(int64_t s, int64_t s_max, int32_t C, int64_t B)
{
    const int64_t by_load = ceil2_ratio(static_cast<u128>(s) * s * C, static_cast<u128>(s_max) * s_max);
    const int64_t by_tokens = ceil2_ratio(static_cast<u128>(s), static_cast<u128>(B));
    return static_cast<int32_t>(std::min<int64_t>(C, std::max(by_load, by_tokens)));
}

struct Group {
    int32_t size;          // ranks
    int32_t opened;        // order of opening inside the micro-batch
    int64_t load_n;        // sum of s^2 of its documents; per-rank load = load_n / size
    int64_t tok_n;         // sum of s; per-rank tokens = tok_n / size
    uint32_t version;      // bumped at every placement: older heap entries are stale
    bool in_capacity_heap; // demoted: token budget too tight for the last document that looked
    int32_t first_doc, last_doc;   // singly linked list of its documents
};

struct LoadEntry { int64_t load_n; int32_t opened; int32_t gid; uint32_t version; };
struct LoadGreater {
    bool operator()(const LoadEntry& a, const LoadEntry& b) const {
        if (a.load_n != b.load_n) return a.load_n > b.load_n;
        return a.opened > b.opened;
    }
};
struct CapEntry { int64_t remaining; int32_t gid; uint32_t version; };
struct CapLess {
    bool operator()(const CapEntry& a, const CapEntry& b) const { return a.remaining < b.remaining; }
};
// per-rank load of a group as the fraction load_n / size
struct RankLoad { int64_t load_n; int32_t size; int32_t opened; int32_t gid; uint32_t version; };
inline bool rank_load_less(int64_t la, int32_t sa, int64_t lb, int32_t sb)
{
    return static_cast<u128>(la) * sb < static_cast<u128>(lb) * sa;
}
struct RankLoadGreater {      // min-heap by per-rank load
    bool operator()(const RankLoad& a, const RankLoad& b) const {
        if (rank_load_less(b.load_n, b.size, a.load_n, a.size)) return true;
        if (rank_load_less(a.load_n, a.size, b.load_n, b.size)) return false;
        return a.opened > b.opened;
    }
};
struct BackfillEntry { int32_t size; int64_t load_n; int32_t opened; int32_t gid; };
struct BackfillGreater {      // min-heap: smallest size, then higher per-rank load, then opened first
    bool operator()(const BackfillEntry& a, const BackfillEntry& b) const {
        if (a.size != b.size) return a.size > b.size;
        if (rank_load_less(a.load_n, a.size, b.load_n, b.size)) return true;     // a lighter: b first
        if (rank_load_less(b.load_n, b.size, a.load_n, a.size)) return false;
        return a.opened > b.opened;
    }
};

struct SizeClass {
    std::priority_queue<LoadEntry, std::vector<LoadEntry>, LoadGreater> by_load;
    std::priority_queue<CapEntry, std::vector<CapEntry>, CapLess> by_capacity;
};

}  // namespace

extern "C" {

int32_t hydra_sched_targets(const int64_t* lengths, int32_t n, int32_t G, int64_t B, int32_t pp,
                            double theta_over_c, hydra_sched_targets_t* out)
{
    if (!lengths || !out || n < 1 || !is_pow2(G) || B < 1 || pp < 1 || !(theta_over_c >= 0.0) ||
        !std::isfinite(theta_over_c))
        return HYDRA_ERR_INVALID_ARG;
    u128 W = 0;
    int64_t s_max = 0;
    for (int32_t i = 0; i < n; ++i) {
        if (lengths[i] < 1) return HYDRA_ERR_INVALID_ARG;
        W += static_cast<u128>(lengths[i]) * lengths[i];
        s_max = std::max(s_max, lengths[i]);
    }
    const double Wd = static_cast<double>(W);
    const double s2 = static_cast<double>(s_max) * static_cast<double>(s_max);
    out->s_max = s_max;
    out->W = Wd;
    out->C_mem = static_cast<int32_t>(std::min<int64_t>(ceil2_ratio(s_max, B), int64_t{1} << 30));
    out->C_hat = s2 * std::sqrt((pp - 1) * theta_over_c * G / Wd);
    int64_t want = out->C_mem;
    if (out->C_hat > static_cast<double>(want)) {
        want = 1;
        while (static_cast<double>(want) < out->C_hat && want < G) want <<= 1;
    }
    out->C_star = static_cast<int32_t>(std::min<int64_t>(G, want));
    out->Lambda_star = s2 / out->C_star;
    const u128 den = static_cast<u128>(G) * s_max * s_max;
    out->M_star = static_cast<int64_t>((static_cast<u128>(out->C_star) * W + den - 1) / den);
    return HYDRA_OK;
}

int32_t hydra_sched_cp(int64_t s, int64_t s_max, int32_t C, int64_t B)
{
    if (s < 1 || s > s_max || !is_pow2(C) || B < 1) return 0;
    return cp_degree(s, s_max, C, B);
}

int32_t hydra_sched_pack(const int64_t* lengths, int32_t n, int32_t G, int64_t B, int32_t C,
                         int32_t* mb_out, int32_t* rank0_out, int32_t* cp_out, int32_t* n_mb_out)
{
    if (!lengths || !mb_out || !rank0_out || !cp_out || !n_mb_out || n < 1 || !is_pow2(G) || !is_pow2(C) ||
        C > G || B < 1)
        return HYDRA_ERR_INVALID_ARG;
    int64_t s_max = 0;
    for (int32_t i = 0; i < n; ++i) {
        if (lengths[i] < 1) return HYDRA_ERR_INVALID_ARG;
        s_max = std::max(s_max, lengths[i]);
    }
    if (static_cast<u128>(C) * B < static_cast<u128>(s_max)) return HYDRA_ERR_INVALID_ARG;   // C below C_mem
    const u128 cap_load_unit = static_cast<u128>(s_max) * s_max;   // Lambda * C

    std::vector<int32_t> order(n);
    for (int32_t i = 0; i < n; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return lengths[a] > lengths[b]; });
    std::vector<int32_t> next_doc(n, -1);

    const int n_classes = log2i(G) + 1;
    int32_t pos = 0, m = 0;
    std::vector<Group> groups;
    while (pos < n) {
        // ---- open a micro-batch over all G ranks
        groups.clear();
        std::vector<SizeClass> classes(n_classes);
        std::priority_queue<RankLoad, std::vector<RankLoad>, RankLoadGreater> lightest;   // lazy, all groups
        int64_t max_load_n = 0;
        int32_t max_size = 1;                       // per-rank maximum max_load_n / max_size
        int32_t free_ranks = G;

        auto feasible_group = [&](int64_t s, int32_t k) -> int32_t {
            const u128 s2 = static_cast<u128>(s) * s;
            for (int j = log2i(k); j < n_classes; ++j) {
                SizeClass& cls = classes[j];
                const int64_t size = int64_t{1} << j;
                // documents arrive longest first: a group whose token budget was too tight for an
                // earlier one may fit this one; re-admit those with enough remaining capacity
                while (!cls.by_capacity.empty()) {
                    const CapEntry top = cls.by_capacity.top();
                    Group& g = groups[top.gid];
                    if (top.version != g.version || !g.in_capacity_heap) { cls.by_capacity.pop(); continue; }
                    if (top.remaining < s) break;
                    cls.by_capacity.pop();
                    g.in_capacity_heap = false;
                    cls.by_load.push(LoadEntry{g.load_n, g.opened, top.gid, g.version});
                }
                while (!cls.by_load.empty()) {
                    const LoadEntry top = cls.by_load.top();
                    Group& g = groups[top.gid];
                    if (top.version != g.version || g.in_capacity_heap || g.size != size) { cls.by_load.pop(); continue; }
                    // the least-loaded group of the class is over the target: so is every other one
                    if ((static_cast<u128>(g.load_n) + s2) * C > cap_load_unit * static_cast<u128>(size)) break;
                    if (static_cast<u128>(g.tok_n) + s > static_cast<u128>(B) * size) {
                        cls.by_load.pop();            // demote: it waits in the capacity heap for a shorter document
                        g.in_capacity_heap = true;
                        cls.by_capacity.push(CapEntry{B * size - g.tok_n, top.gid, g.version});
                        continue;
                    }
                    return top.gid;
                }
            }
            return -1;
        };

        while (pos < n) {
            const int32_t i = order[pos];
            const int64_t s = lengths[i];
            const int32_t k = cp_degree(s, s_max, C, B);
            int32_t gid;
            if (free_ranks >= k) {
                gid = static_cast<int32_t>(groups.size());
                groups.push_back(Group{k, gid, 0, 0, 0u, false, -1, -1});
                free_ranks -= k;
            } else {
                gid = feasible_group(s, k);
                if (gid < 0) break;
            }
            Group& g = groups[gid];
            if (g.first_doc < 0) g.first_doc = i; else next_doc[g.last_doc] = i;
            g.last_doc = i;
            g.load_n += s * s;
            g.tok_n += s;
            ++g.version;
            classes[log2i(g.size)].by_load.push(LoadEntry{g.load_n, g.opened, gid, g.version});
            lightest.push(RankLoad{g.load_n, g.size, g.opened, gid, g.version});
            if (rank_load_less(max_load_n, max_size, g.load_n, g.size)) { max_load_n = g.load_n; max_size = g.size; }
            ++pos;
            // early-close test of Algorithm 1, Phase 2: the next document needs a smaller degree, no rank is
            // free, and the micro-batch is balanced
            if (pos < n && free_ranks == 0 && cp_degree(lengths[order[pos]], s_max, C, B) < k) {
                while (lightest.top().version != groups[lightest.top().gid].version) lightest.pop();
                const RankLoad lo = lightest.top();
                // 4 * lo >= 3 * hi on per-rank loads
                if (!(static_cast<u128>(4) * lo.load_n * max_size < static_cast<u128>(3) * max_load_n * lo.size)) break;
            }
        }
        // ---- backfill idle ranks by doubling the smallest group
        if (free_ranks > 0 && !groups.empty()) {
            std::priority_queue<BackfillEntry, std::vector<BackfillEntry>, BackfillGreater> smallest;
            for (int32_t gid = 0; gid < static_cast<int32_t>(groups.size()); ++gid)
                smallest.push(BackfillEntry{groups[gid].size, groups[gid].load_n, groups[gid].opened, gid});
            while (true) {
                const BackfillEntry top = smallest.top();
                if (top.size > free_ranks) break;
                smallest.pop();
                free_ranks -= top.size;
                groups[top.gid].size = top.size * 2;
                smallest.push(BackfillEntry{top.size * 2, top.load_n, top.opened, top.gid});
            }
        }
        // ---- ranks: groups in order of decreasing size take consecutive (hence aligned) blocks
        std::vector<int32_t> by_size(groups.size());
        for (size_t gi = 0; gi < groups.size(); ++gi) by_size[gi] = static_cast<int32_t>(gi);
        std::stable_sort(by_size.begin(), by_size.end(),
                         [&](int32_t a, int32_t b) { return groups[a].size > groups[b].size; });
        int32_t at = 0;
        for (int32_t gid : by_size) {
            const Group& g = groups[gid];
            for (int32_t d = g.first_doc; d >= 0; d = next_doc[d]) {
                mb_out[d] = m;
                rank0_out[d] = at;
                cp_out[d] = g.size;
            }
            at += g.size;
        }
        ++m;
    }
    *n_mb_out = m;
    return HYDRA_OK;
}

}  // extern "C"
