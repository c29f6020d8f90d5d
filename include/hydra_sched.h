/*
 * hydra_sched.h - the load-driven dynamic-context-parallel scheduler (Section 5.1), host only.
 *
 * The attention entry points of hydra_attn.h take chunk pairs; this is the step before them: it
 * decides, for a batch of documents and a pool of G ranks, which micro-batch (MB) every document
 * goes to and on how many ranks it runs (its CP degree). The degree then factors into an inner
 * Ulysses group and an outer ring with hydra_usp_factor, and the ring factor cuts the document into
 * the zigzag chunk pairs of hydra_zigzag_pairs.
 *
 * Everything here runs on the host; all pointers are host memory owned by the caller; no call
 * touches a GPU. Status codes are those of hydra_attn.h.
 */
#ifndef HYDRA_SCHED_H
#define HYDRA_SCHED_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif
#if defined(__GNUC__)
#pragma GCC visibility push(default)
#endif

/*
 * Closed-form targets (Section 5.1.1). For document lengths s_i, pool size G, per-rank token budget
 * B, pipeline depth pp and the measured ratio theta / c (time per unit of per-rank load over the
 * fixed cost of a micro-batch):
 *   W        = sum s_i^2                                              (total quadratic work)
 *   C_mem    = ceil2(s_max / B)                                        (Eq. cstar)
 *   C_hat    = s_max^2 sqrt((pp - 1) (theta / c) G / W)                (Eq. cstar-cont)
 *   C_star   = min{G, ceil2(max{C_mem, C_hat})}                        (Eq. cstar)
 *   Lambda   = s_max^2 / C_star                                        (Eq. load-target)
 *   M_star   = ceil(C_star W / (G s_max^2))                            (Eq. mstar)
 * ceil2(x) is the smallest power of two that is at least x. W is returned as a double (exact below
 * 2^53); M_star is computed exactly in integers.
 * Errors: HYDRA_ERR_INVALID_ARG for n < 1, a length < 1, G not a power of two, B < 1, pp < 1 or a
 * negative or non-finite theta_over_c.
 */
typedef struct {
    int64_t s_max;
    double W;
    int32_t C_mem;
    int32_t C_star;
    double C_hat;
    double Lambda_star;
    int64_t M_star;
} hydra_sched_targets_t;

int32_t hydra_sched_targets(const int64_t* lengths, int32_t n, int32_t G, int64_t B, int32_t pp,
                            double theta_over_c, hydra_sched_targets_t* out);

/*
 * CP degree of a document of length s (Eq. cp): the smallest power of two that keeps its per-rank
 * load within Lambda = s_max^2 / C and its per-rank tokens within B, capped at C:
 *   cp(s) = min{C, ceil2(max{s^2 / Lambda, s / B})},
 * evaluated in exact integer arithmetic. Returns the degree, or 0 on invalid arguments (s < 1,
 * s > s_max, C not a power of two, B < 1).
 */
int32_t hydra_sched_cp(int64_t s, int64_t s_max, int32_t C, int64_t B);

/*
 * Algorithm 1 (longest-first piggyback packing, Sections 5.1.2 and 5.1.3). Documents are taken
 * longest first (equal lengths in input order), one micro-batch at a time over all G ranks:
 *   - a document of degree k = cp(s) opens a new group of k ranks while k ranks are free;
 *   - otherwise it joins the smallest open group of at least k ranks that stays within the load
 *     target (load + s^2 / |g| <= Lambda) and the token budget (tokens + s / |g| <= B), the less
 *     loaded one among equals, the one opened first among those;
 *   - if there is none, the micro-batch is closed and the document opens the next one;
 *   - the micro-batch is also closed when the next document's degree is smaller than the one just
 *     used, no rank is free, and the least-loaded group carries at least 3/4 of the per-rank load
 *     of the most loaded one (the early-close test at the end of Algorithm 1's inner loop, which the
 *     paper names without defining it: this is the reading taken here);
 *   - idle ranks of a closed micro-batch are backfilled by doubling the smallest group (the more
 *     loaded one among equals) while it is no larger than the number of idle ranks;
 *   - groups then take consecutive rank blocks in order of decreasing size, so that every group
 *     sits on a block aligned to its own size.
 * The search keeps, per group size, a lazy min-heap by load and a max-heap by remaining token
 * capacity (Section 5.1.3): O(N log G) instead of a scan of every open group per document, with
 * exactly the placements of the scan.
 *   lengths[n]   host, document lengths (tokens), each in [1, C * B]
 *   G, C         powers of two, C <= G; C * B >= max length
 *   mb_out[n]    micro-batch of document i
 *   rank0_out[n] first rank of its group inside the micro-batch
 *   cp_out[n]    number of ranks of its group (>= cp(s_i); larger after backfill)
 *   n_mb_out     number of micro-batches (the value the paper broadcasts to the pipeline stages)
 * Errors: HYDRA_ERR_INVALID_ARG for null pointers or arguments outside the ranges above.
 */
int32_t hydra_sched_pack(const int64_t* lengths, int32_t n, int32_t G, int64_t B, int32_t C,
                         int32_t* mb_out, int32_t* rank0_out, int32_t* cp_out, int32_t* n_mb_out);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif
#ifdef __cplusplus
}
#endif
#endif
