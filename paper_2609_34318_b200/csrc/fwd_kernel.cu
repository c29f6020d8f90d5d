// Forward attention of (q-chunk, kv-chunk) pairs on sm_100a, on CTA PAIRS (cluster of two,
// tcgen05 cta_group::2).
//
// A work item is a 512-row slab of q rows of one pair and head, handled by one CTA pair as two
// 256-row UMMA tiles (A and B); each CTA owns 128 rows of each tile. The two tiles ping-pong on the
// tensor cores so that the UMMAs of one overlap the softmax of the other. Every K/V tile is fetched
// from L2 once per pair and each CTA stages only its half of it (64 kv rows of K for S = Q K^T, 64
// value columns of V for O += P V), so three stages of K and of V fit next to the two Q tiles: deep
// enough to cover the latency of a TMA load, which two full-size stages could not.
//
// Warp roles per CTA (352 threads):
//   warps 0-3   softmax of this CTA's rows of tile A: thread r owns row r = TMEM lane r
//   warps 4-7   softmax of this CTA's rows of tile B
//   warp  8     TMA producer of Q (per item) and K
//   warp  9     TMA producer of V
//   warp 10     leader CTA only: UMMA issuer (one thread); both CTAs: TMEM allocation
// Barriers live at the same shared-memory offsets in both CTAs. "Full" barriers are used in the
// leader's copy (both CTAs' TMA loads count their bytes there; both CTAs' softmax warps arrive
// there); "done" events of the tensor core are committed to both copies at once.
//
// Tensor memory (512 columns per CTA): S_A [0,128) S_B [128,256) O_A [256,384) O_B [384,512); P (bf16
// pairs) is written over the first 64 columns of its S. Issue order per kv tile j:
//   S_A(j) = Q_A K_j^T ; O_B += P_B(j-1) V_{j-1} ; S_B(j) = Q_B K_j^T ; O_A += P_A(j) V_j
// The softmax keeps a running maximum in the exp2 domain and rescales O only when the maximum grew
// by more than 2^8 (the final LSE is exact whatever reference maximum was used).
// Items come from a run-time queue: the leader's producer pops an index from a counter in global
// memory and hands it to every other role of both CTAs through a ring in (distributed) shared memory.
#include <cuda_bf16.h>

#include "hydra_internal.h"
#include "sm100_ptx.cuh"

// This file is compiled once per supported q / k head dimension (HYDRA_KERNEL_DQK = 192, the default, or
// 128); the value dimension is 128 in both. HYDRA_K() gives the kernels and launchers of the second
// build their own names.
#ifndef HYDRA_KERNEL_DQK
#define HYDRA_KERNEL_DQK 192
#endif
#if HYDRA_KERNEL_DQK == 192
#define HYDRA_K(name) name
#elif HYDRA_KERNEL_DQK == 128
#define HYDRA_K(name) name##_d128
#else
#error "unsupported q / k head dimension"
#endif

namespace hydra {

namespace {

constexpr int kDqk = HYDRA_KERNEL_DQK;
constexpr int kQkBoxes = kDqk / 64;                    // 64-column boxes of a q / k row
constexpr int kThreads = 352;
constexpr int kWarpK = 8, kWarpV = 9, kWarpMma = 10;
constexpr uint32_t kBox = 128 * 128;                  // [128 rows x 64 bf16] = 16 KB
constexpr uint32_t kHalfBox = 64 * 128;               // [ 64 rows x 64 bf16] =  8 KB
constexpr uint32_t kQTile = kQkBoxes * kBox;          // this CTA's 128 rows of a q tile
constexpr uint32_t kKStage = kQkBoxes * kHalfBox;     // this CTA's 64 kv rows of a k tile
constexpr uint32_t kVStage = kBox;                    // 128 kv rows x this CTA's 64 value columns
constexpr int kKStages = 3, kVStages = 3;
constexpr uint32_t kSmemQ = 0;
constexpr uint32_t kSmemK = kSmemQ + 2 * kQTile;
constexpr uint32_t kSmemV = kSmemK + kKStages * kKStage;
constexpr uint32_t kSmemTotal = kSmemV + kVStages * kVStage;  // 221,184 B at d_qk = 192
constexpr uint32_t kTmS = 0, kTmO = 256, kTmCols = 512;
constexpr float kRescaleThreshold = 8.f;              // log2 units

constexpr int kSched = 4;                             // depth of the in-cluster ring of work-item indices

enum : int {
    B_QFULL = 0, B_QEMPTY = 2, B_KFULL = 4, B_KEMPTY = 7, B_VFULL = 10, B_VEMPTY = 13,
    B_SFULL = 16, B_PFULL = 18, B_OFULL = 20, B_OFREE = 22, B_PFULL2 = 24,
    B_ITEMFULL = 26, B_ITEMEMPTY = 26 + kSched, B_COUNT = 26 + 2 * kSched
};

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

}  // namespace

size_t HYDRA_K(fwd_smem_bytes)() { return kSmemTotal + 1024; }

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
HYDRA_K(hydra_fwd_kernel)(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const FwdParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem = (smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t bars[B_COUNT];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ int32_t s_sched[kSched];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_cta_rank();
    const bool leader = rank == 0;
    const uint32_t bar0 = smem_u32(&bars[0]);
    auto bar = [&](int i) -> uint32_t { return bar0 + 8u * static_cast<uint32_t>(i); };

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < B_COUNT; ++i) {
            // P-ready and O-drained collect the 4 softmax warps of a tile in each of the 2 CTAs
            const bool by_warps = (i >= B_PFULL && i < B_PFULL + 2) || (i >= B_OFREE && i < B_OFREE + 2) ||
                                  (i >= B_PFULL2 && i < B_PFULL2 + 2);
            // an item slot is free again when every reader of both CTAs has taken the index: 8 softmax
            // warps and 2 single-thread roles per CTA
            const bool by_readers = i >= B_ITEMEMPTY && i < B_ITEMEMPTY + kSched;
            mbar_init(bar(i), by_readers ? 20u : (by_warps ? 8u : 1u));
        }
        fence_mbar_init();
        tma_prefetch_desc(&map_q); tma_prefetch_desc(&map_k); tma_prefetch_desc(&map_v);
    }
    if (warp == kWarpMma) { tmem_alloc_pair(smem_u32(&tmem_base_slot), kTmCols); tmem_relinquish_pair(); }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                                // both CTAs' barriers exist before anyone signals them
    tc_fence_after_sync();
    const uint32_t tm = tmem_base_slot;
    const uint64_t limit = p.wait_limit_ns;
    volatile int* abort_p = &abort_flag;
    auto wait = [&](int b, uint32_t parity) -> bool { return mbar_wait(bar(b), parity & 1u, abort_p, limit); };
    // Work queue: the leader's producer pops the next item index from a counter in global memory (a
    // cluster that finishes early simply takes more items: no cost model has to predict the run time
    // of an item) and hands it to every other role of both CTAs through a small ring that exists in
    // both CTAs' shared memory.
    volatile int32_t* sched = s_sched;
    auto pop_item = [&](uint32_t k) -> int {                 // leader CTA, one thread
        const int slot = k % kSched;
        if (!mbar_wait(bar(B_ITEMEMPTY + slot), ((k / kSched) ^ 1u) & 1u, abort_p, limit)) return -1;
        int idx = atomicAdd(&p.status->next_item[QUEUE_FWD], 1);
        if (idx >= p.n_items) idx = -1;
        for (uint32_t r = 0; r < 2; ++r) {
            st_shared_cluster_s32(cluster_map_shared(smem_u32(&s_sched[slot]), r), idx);
            mbar_arrive_cluster_release(cluster_map_shared(bar(B_ITEMFULL + slot), r));
        }
        return idx;
    };
    auto next_item = [&](uint32_t k, bool whole_warp) -> int {   // every other role, either CTA
        const int slot = k % kSched;
        if (!mbar_wait_acquire_cluster(bar(B_ITEMFULL + slot), (k / kSched) & 1u, abort_p, limit)) return -1;
        const int idx = sched[slot];
        if (whole_warp) mbar_arrive_warp_leader(bar(B_ITEMEMPTY + slot));
        else mbar_arrive_leader(bar(B_ITEMEMPTY + slot));
        return idx;
    };

    if (warp == kWarpK) {
        // ------------------------------------------------------------------ Q and K producer
        if (lane == 0) {
            uint32_t gk = 0, q_use[2] = {0, 0};
            bool ok = true;
            ClockProbe probe;
            probe.start();
            // test hook: idle, then hand out and load nothing; every other role's wait then runs out
            if (p.debug_stall_ns) { debug_stall(p.debug_stall_ns); ok = false; }
            // the leader pops one item ahead: the round trip to the counter and the hand-over to the
            // other CTA then overlap the loads of the current item
            int it_ahead = (leader && ok) ? pop_item(0) : 0;
            for (uint32_t kq = 0; ok; ++kq) {
                int it;
                if (leader) {
                    it = it_ahead;
                    if (it >= 0) it_ahead = pop_item(kq + 1);
                } else {
                    it = next_item(kq, false);
                }
                if (it < 0) break;
                const FwdItem item = p.items[it];
                const PairDev pr = p.pairs[item.pair];
                const int n_t[2] = {item.n_a, item.n_b};
                const int n = max(item.n_a, item.n_b);
                auto load_q = [&](int t) {
                    if (n_t[t] <= 0 || !ok) return;
                    ok = wait(B_QEMPTY + t, q_use[t] ^ 1u);
                    if (!ok) return;
                    ++q_use[t];
                    if (leader) mbar_arrive_expect_tx(bar(B_QFULL + t), 2 * kQTile);
                    for (int c = 0; c < kQkBoxes; ++c)
                        tma_load_3d_pair(smem + kSmemQ + t * kQTile + c * kBox, &map_q, bar(B_QFULL + t), c * 64,
                                         item.head, pr.q_tok0 + item.q0 + t * 2 * TILE + rank * TILE);
                };
                auto load_k = [&](int j) {
                    const int slot = gk % kKStages;
                    ok = wait(B_KEMPTY + slot, (gk / kKStages) ^ 1u);
                    if (!ok) return;
                    ++gk;
                    if (leader) mbar_arrive_expect_tx(bar(B_KFULL + slot), 2 * kKStage);
                    for (int c = 0; c < kQkBoxes; ++c)
                        tma_load_3d_pair(smem + kSmemK + slot * kKStage + c * kHalfBox, &map_k, bar(B_KFULL + slot),
                                         c * 64, item.head / p.kv_group, pr.k_tok0 + j * TILE + rank * 64);
                };
                // The Q buffer of tile B is released by the very last score product of the previous item,
                // the K stages one and two tiles earlier: ask for the first K tiles before waiting for it.
                load_q(0);
                int j = 0;
                for (; j < n && j < kKStages - 1 && ok; ++j) load_k(j);
                load_q(1);
                for (; j < n && ok; ++j) load_k(j);
            }
            if (blockIdx.x == 0) probe.stop(p.status, QUEUE_FWD);
        }
    } else if (warp == kWarpV) {
        // ------------------------------------------------------------------ V producer
        if (lane == 0) {
            uint32_t gv = 0;
            bool ok = true;
            for (uint32_t kq = 0; ok; ++kq) {
                const int it = next_item(kq, false);
                if (it < 0) break;
                const FwdItem item = p.items[it];
                const PairDev pr = p.pairs[item.pair];
                const int n = max(item.n_a, item.n_b);
                for (int j = 0; j < n && ok; ++j, ++gv) {
                    const int slot = gv % kVStages;
                    ok = wait(B_VEMPTY + slot, (gv / kVStages) ^ 1u);
                    if (!ok) break;
                    if (leader) mbar_arrive_expect_tx(bar(B_VFULL + slot), 2 * kVStage);
                    tma_load_3d_pair(smem + kSmemV + slot * kVStage, &map_v, bar(B_VFULL + slot), rank * 64,
                                     item.head / p.kv_group, pr.k_tok0 + j * TILE);
                }
            }
        }
    } else if (warp == kWarpMma) {
        // ------------------------------------------------------------------ UMMA issuer (leader CTA)
        if (leader && elect_one()) {
            constexpr uint32_t idesc_s = umma_idesc_bf16(2 * TILE, TILE, false, false);
            constexpr uint32_t idesc_o = umma_idesc_bf16(2 * TILE, D_V, false, true);
            constexpr uint32_t hi_k = umma_desc_hi(16, 1024);           // K-major Q and K boxes
            constexpr uint32_t hi_v = umma_desc_hi(kBox, 1024);         // MN-major V (one 64-column chunk)
            const uint32_t q_lo[2] = {umma_desc_lo(smem + kSmemQ, 16), umma_desc_lo(smem + kSmemQ + kQTile, 16)};
            const uint32_t k_lo0 = umma_desc_lo(smem + kSmemK, 16);
            const uint32_t v_lo0 = umma_desc_lo(smem + kSmemV, kBox);
            uint32_t ks = 0, kp = 0;                 // stage / phase of kv tile j in the K ring
            uint32_t vs = 0, vp = 0, vs_prev = 0, vp_prev = 0;   // same for V, tiles j and j-1
            uint32_t q_use[2] = {0, 0}, c_p[2] = {0, 0}, free_use[2] = {0, 0};
            bool ok = true;
            for (uint32_t kq = 0; ok; ++kq) {
                const int it = next_item(kq, false);
                if (it < 0) break;
                const FwdItem item = p.items[it];
                const int n_t[2] = {item.n_a, item.n_b};
                const int n = max(item.n_a, item.n_b);

                // One step of a tile's chain: finish kv tile `jpv` (O += P V) and start kv tile `js`
                // (S = Q K^T), back to back. The polls that are almost always satisfied (K, V, Q
                // landed; O drained) come first, so that once the softmax has delivered P nothing
                // but UMMAs and commits stands between the end of one product and the start of the
                // next: the tile's chain S -> softmax -> P V -> S is the critical path.
                auto advance = [&](int t, int jpv, uint32_t v_slot, uint32_t v_ph, int js, uint32_t k_slot,
                                   uint32_t k_ph) {
                    const bool do_pv = jpv >= 0 && jpv < n_t[t];
                    const bool do_s = js < n_t[t];
                    if (do_s) {
                        if (js == 0) {
                            ok = wait(B_QFULL + t, q_use[t]);
                            ++q_use[t];
                            if (!ok) return;
                        }
                        ok = wait(B_KFULL + k_slot, k_ph);
                        if (!ok) return;
                    }
                    const uint32_t d_s = tm + kTmS + t * TILE, d_o = tm + kTmO + t * D_V;
                    if (do_pv) {
                        ok = wait(B_VFULL + v_slot, v_ph);
                        if (!ok) return;
                        if (jpv == 0) {
                            ok = wait(B_OFREE + t, free_use[t] ^ 1u);
                            ++free_use[t];
                            if (!ok) return;
                        }
                        // P arrives in two instalments (columns [0,64) and [64,128)): the first half of
                        // the product runs while the second half of the exponentials is being computed
                        ok = wait(B_PFULL + t, c_p[t]);
                        if (!ok) return;
                        tc_fence_after_sync();
                        const uint32_t b_lo = v_lo0 + v_slot * (kVStage >> 4);
#pragma unroll
                        for (int kk = 0; kk < TILE / 32; ++kk)
                            umma2_ts_w(d_o, d_s + kk * 8, b_lo + kk * (2048 >> 4), hi_v, idesc_o, (jpv | kk) != 0);
                        ok = wait(B_PFULL2 + t, c_p[t]);
                        ++c_p[t];
                        if (!ok) return;
                        tc_fence_after_sync();
#pragma unroll
                        for (int kk = TILE / 32; kk < TILE / 16; ++kk)
                            umma2_ts_w(d_o, d_s + kk * 8, b_lo + kk * (2048 >> 4), hi_v, idesc_o, 1u);
                        if ((t == 1) || (jpv >= n_t[1])) umma2_commit(bar(B_VEMPTY + v_slot));   // last reader
                        umma2_commit(bar(B_OFULL + t));
                    } else {
                        tc_fence_after_sync();
                    }
                    if (do_s) {
                        const uint32_t b_lo = k_lo0 + k_slot * (kKStage >> 4);
#pragma unroll
                        for (int kk = 0; kk < kDqk / 16; ++kk)
                            umma2_ss_w(d_s, q_lo[t] + (kk >> 2) * (kBox >> 4) + (kk & 3) * 2, hi_k,
                                       b_lo + (kk >> 2) * (kHalfBox >> 4) + (kk & 3) * 2, hi_k, idesc_s, kk != 0);
                        if ((t == 1) || (js >= n_t[1])) umma2_commit(bar(B_KEMPTY + k_slot));    // last reader
                        umma2_commit(bar(B_SFULL + t));
                        if (js == n_t[t] - 1) umma2_commit(bar(B_QEMPTY + t));
                    }
                };

                // issue order: S_A(0) | S_B(0) | PV_A(0) S_A(1) | PV_B(0) S_B(1) | PV_A(1) S_A(2) | ...
                advance(0, -1, 0u, 0u, 0, ks, kp);
                for (int j = 0; j <= n && ok; ++j) {
                    uint32_t ks1 = ks + 1u, kp1 = kp;          // ring position of kv tile j + 1
                    if (ks1 == kKStages) { ks1 = 0; kp1 ^= 1u; }
                    advance(1, j - 1, vs_prev, vp_prev, j, ks, kp);
                    if (ok) advance(0, j, vs, vp, j + 1, ks1, kp1);
                    if (j < n) {                     // step the ring cursors to kv tile j + 1
                        vs_prev = vs; vp_prev = vp;
                        ks = ks1; kp = kp1;
                        if (++vs == kVStages) { vs = 0; vp ^= 1u; }
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax warpgroups
        const int t = warp >> 2;                       // tile A or B
        const int r = tid & 127;                       // row inside this CTA's half of the tile = TMEM lane
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tm_s = tm + kTmS + t * TILE + lane_base;
        const uint32_t tm_o = tm + kTmO + t * D_V + lane_base;
        uint32_t c_s = 0, c_o = 0;
        bool ok = true;
        for (uint32_t kq = 0; ok; ++kq) {
            const int it = next_item(kq, true);
            if (it < 0) break;
            const FwdItem item = p.items[it];
            const PairDev pr = p.pairs[item.pair];
            const int n_kv = t == 0 ? item.n_a : item.n_b;
            const int row0 = item.q0 + t * 2 * TILE + static_cast<int>(rank) * TILE;   // first row of this CTA
            const int row = row0 + r;                  // q row inside the pair
            const bool row_valid = row < pr.q_len;
            const int64_t rows_total = pr.to_part ? p.part_rows : p.T;
            __nv_bfloat16* obase = static_cast<__nv_bfloat16*>(pr.to_part ? p.o_part : p.out);
            float* lbase = pr.to_part ? p.lse_part : p.lse;
            const int64_t orow = static_cast<int64_t>(pr.out_row0) + row;
            uint4* dst = reinterpret_cast<uint4*>(obase + (orow * p.h + item.head) * D_V);
            float* lse_dst = lbase + static_cast<int64_t>(item.head) * rows_total + orow;

            if (n_kv <= 0) {                           // rows that see no key: O = 0, LSE = -inf
                if (row_valid && n_kv == 0) {           // (n_kv < 0: no such tile in this item)
#pragma unroll
                    for (int e = 0; e < D_V / 8; ++e) dst[e] = make_uint4(0u, 0u, 0u, 0u);
                    *lse_dst = neg_inf();
                }
                continue;
            }
            float m_run = neg_inf(), l_run = 0.f;
            for (int j = 0; j < n_kv && ok; ++j) {
                ok = wait(B_SFULL + t, c_s);
                ++c_s;
                if (!ok) break;
                tc_fence_after_sync();
                const int col0 = j * TILE;
                const bool need_mask = (col0 + TILE > pr.k_len) || (p.causal && (col0 + TILE - 1 > row0 + pr.off));
                int cmax = TILE;                       // columns 0..cmax are visible
                if (need_mask) {
                    int jmax = pr.k_len - 1;
                    if (p.causal) jmax = min(jmax, row + pr.off);
                    cmax = jmax - col0;
                }
                // pass 1: row maximum, 64 columns at a time (the 168 registers a thread may use do not
                // hold a whole row of S next to the probabilities without spilling)
                float mx0 = neg_inf(), mx1 = neg_inf(), mx2 = neg_inf(), mx3 = neg_inf();
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t s[TILE / 2];
                    tmem_ld_x32(tm_s + half * 64, s);
                    tmem_ld_x32(tm_s + half * 64 + 32, s + 32);
                    tmem_wait_ld();
                    if (need_mask) {
#pragma unroll
                        for (int c = 0; c < TILE / 2; ++c)
                            if (half * 64 + c > cmax) s[c] = __float_as_uint(neg_inf());
                    }
#pragma unroll
                    for (int c = 0; c < TILE / 2; c += 8) {
                        mx0 = fmax3(mx0, __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
                        mx1 = fmax3(mx1, __uint_as_float(s[c + 2]), __uint_as_float(s[c + 3]));
                        mx2 = fmax3(mx2, __uint_as_float(s[c + 4]), __uint_as_float(s[c + 5]));
                        mx3 = fmax3(mx3, __uint_as_float(s[c + 6]), __uint_as_float(s[c + 7]));
                    }
                }
                const float m_new = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2;
                float alpha = 1.f;
                if (m_new > m_run + kRescaleThreshold || (j == 0)) {
                    alpha = ex2_approx(m_run - m_new);          // 0 when m_run = -inf
                    if (m_new == neg_inf()) alpha = 1.f;         // nothing visible yet: keep -inf
                    else m_run = m_new;
                }
                const float m_use = (m_run == neg_inf()) ? 0.f : m_run;
                if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                    // Rescale O before any part of this tile's product is added to it. The previous
                    // P V of this tile has landed: it was issued before this tile's S, which has
                    // completed, and the tensor pipe runs in issue order.
#pragma unroll
                    for (int c0 = 0; c0 < D_V; c0 += 32) {
                        uint32_t o[32];
                        tmem_ld_x32(tm_o + c0, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                        tmem_st_x32(tm_o + c0, o);
                    }
                }
                // pass 2: P = exp2(S * c - m) as packed bf16, written over the first half of S and handed
                // to the tensor core in two instalments (columns [0,64), then [64,128)).
                float rs0 = 0.f, rs1 = 0.f;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t s[TILE / 2], pk[TILE / 4];
                    tmem_ld_x32(tm_s + half * 64, s);
                    tmem_ld_x32(tm_s + half * 64 + 32, s + 32);
                    tmem_wait_ld();
                    if (need_mask) {
#pragma unroll
                        for (int c = 0; c < TILE / 2; c += 2) {
                            float p0 = ex2_approx(fmaf(__uint_as_float(s[c]), p.scale_log2, -m_use));
                            float p1 = ex2_approx(fmaf(__uint_as_float(s[c + 1]), p.scale_log2, -m_use));
                            if (half * 64 + c > cmax) p0 = 0.f;
                            if (half * 64 + c + 1 > cmax) p1 = 0.f;
                            rs0 += p0;
                            rs1 += p1;
                            pk[c >> 1] = pack_bf16x2(p0, p1);
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < TILE / 2; c += 2) {
                            float x0, x1;
                            ffma2(x0, x1, __uint_as_float(s[c]), __uint_as_float(s[c + 1]), p.scale_log2, p.scale_log2,
                                  -m_use, -m_use);
                            const float p0 = ex2_approx(x0);
                            const float p1 = ex2_approx(x1);
                            fadd2(rs0, rs1, rs0, rs1, p0, p1);
                            pk[c >> 1] = pack_bf16x2(p0, p1);
                        }
                    }
                    tmem_st_x32(tm_s + half * 32, pk);
                    tmem_wait_st();
                    tc_fence_before_sync();
                    mbar_arrive_warp_leader(bar((half == 0 ? B_PFULL : B_PFULL2) + t));
                }
                l_run = l_run * alpha + (rs0 + rs1);
                ++c_o;
            }
            if (!ok) break;
            // ---- epilogue: O / l -> bf16, LSE = ln2 * (m + log2 l) ---------------------------------
            ok = wait(B_OFULL + t, c_o - 1u);
            if (!ok) break;
            tc_fence_after_sync();
            const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
            const bool wide = (reinterpret_cast<uintptr_t>(dst) & 31u) == 0;
#pragma unroll
            for (int c0 = 0; c0 < D_V; c0 += 32) {
                uint32_t o[32];
                tmem_ld_x32(tm_o + c0, o);
                tmem_wait_ld();
                if (c0 + 32 == D_V) {                  // every column has left TMEM: O may be overwritten
                    tc_fence_before_sync();
                    mbar_arrive_warp_leader(bar(B_OFREE + t));
                }
                if (row_valid) {
                    // 32 bytes per store where the address allows it (the interface asks for 16): a thread's row
                    // is 4 KB from its neighbour's, every store of a warp touches 32 lines, whole sectors halve
                    // the number of such instructions
#pragma unroll
                    for (int e = 0; e < 32; e += 16) {
                        uint32_t w[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            w[i] = pack_bf16x2(__uint_as_float(o[e + 2 * i]) * inv_l, __uint_as_float(o[e + 2 * i + 1]) * inv_l);
                        if (wide) {
                            st_global_v8(dst + ((c0 + e) >> 3), w);
                        } else {
                            dst[(c0 + e) >> 3] = make_uint4(w[0], w[1], w[2], w[3]);
                            dst[((c0 + e) >> 3) + 1] = make_uint4(w[4], w[5], w[6], w[7]);
                        }
                    }
                }
            }
            if (row_valid)
                *lse_dst = (l_run > 0.f) ? (m_run + __log2f(l_run)) * 0.6931471805599453f : neg_inf();
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                                // the leader's UMMAs read the peer's memories
    if (abort_flag) {
        // A wait ran out. Give copies still in flight time to land, then report and leave.
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 50000ull) { }
        if (tid == 0) {
            p.status->detail = blockIdx.x;
            p.status->status = HYDRA_ERR_DEVICE_TIMEOUT;
        }
        __syncthreads();
    }
    if (warp == kWarpMma) tmem_dealloc_pair(tm, kTmCols);
}

// Number of CTA pairs that can be resident at once (one CTA per SM): the size of the persistent grid.
// Kept per device ordinal: the shared-memory opt-in applies to the device that is current when it is made.
int HYDRA_K(fwd_max_clusters)()
{
    static int cached_by_device[64];
    static bool known[64] = {};
    int sms = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (known[dev]) return cached_by_device[dev];
    if (cudaFuncSetAttribute(HYDRA_K(hydra_fwd_kernel), cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(HYDRA_K(fwd_smem_bytes)())) != cudaSuccess)
        return 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(sms / 2 * 2));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = HYDRA_K(fwd_smem_bytes)();
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, HYDRA_K(hydra_fwd_kernel), &cfg) != cudaSuccess) n = 0;
    cached_by_device[dev] = n;
    known[dev] = n > 0;
    return n;
}

cudaError_t HYDRA_K(launch_fwd)(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                       const FwdParams& p, int n_clusters, cudaStream_t stream)
{
    HYDRA_K(hydra_fwd_kernel)<<<2 * n_clusters, kThreads, HYDRA_K(fwd_smem_bytes)(), stream>>>(mq, mk, mv, p);
    return cudaGetLastError();
}

}  // namespace hydra
