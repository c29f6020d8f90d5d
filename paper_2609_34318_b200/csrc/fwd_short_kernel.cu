// Forward attention of SHORT (q-chunk, kv-chunk) pairs on sm_100a: one CTA per SM, two independent q tiles
// in flight per CTA.
//
// The paper's workload is dominated by short sequences (Section 2.2). On a 300-token sequence the CTA-pair
// kernel (fwd_kernel.cu) is bound by the LENGTH of a tile's chain S -> softmax -> P V, not by the tensor
// cores: a 512-row slab keeps two SMs busy for three serial steps of 4000-5000 cycles each. What helps there
// is more chains in flight per SM and shorter steps. This kernel therefore gives every SM two SLOTS, each a
// complete pipeline of its own (TMA producer thread, UMMA issuer thread, four softmax warps, 256 columns of
// tensor memory, its own Q tile and K / V rings), working on its own work items: a work item is one 128-row
// q tile of one pair and head, and a step covers 64 keys. Nothing is shared between the slots but the work
// queue, so the tensor pipe always has the other slot's products to run while one slot's softmax is busy.
//
// Per slot, tensor memory holds O [0,128) and TWO score buffers S0 [128,192), S1 [192,256): the score
// product of step j + 1 (and j + 2) is issued before the softmax of step j has finished, so the softmax
// warps never wait for the tensor core inside a work item; P (bf16 pairs) is written over the first 32
// columns of its own S buffer. The steps of consecutive work items form one stream: the producer requests
// the next item's Q and first K tile before the current item's last V tile, and the issuer puts the next
// item's first score products behind the current item's last P V, so the next item's first S is ready when
// the softmax warps come out of the epilogue.
//
// Warp roles (384 threads): warps 0-3 / 4-7 softmax of slot 0 / 1 (thread r = q row r = TMEM lane r),
// warps 8 / 9 producers (one thread each: pops work items from the run-time queue, TMA loads), warps 10 / 11
// UMMA issuers (one thread each; warp 10 also allocates the tensor memory).
// K is staged as [64 keys x d_qk] (K-major B operand of S = Q K^T, N = 64), V as [64 keys x 128] in two
// 64-column boxes (MN-major B operand of O += P V), both straight from their token-major TMA tiles.
//
// What bounds a slot in steady state at d_qk = 192 is its single V stage (V(j + 1) can only be asked for when
// P V(j) has completed and arrives about 1600 cycles later), which is about what the softmax of 64 columns takes
// with its fixed latencies; on a workload of 300-token sequences the kernel as a whole is bound by HBM (it moves
// 5.3 TB/s). Measured and not kept: four more warps that read O out and store it while the softmax warps start
// the next item (512 threads, registers divided with setmaxnreg, row sums handed over in shared memory: 34 %
// slower on short sequences, 9 % on 4096-token ones, although the same kernel with the extra warps idle ran as
// fast as without them); handing P over at the start of the next step, after the next scores have been asked
// for from tensor memory (2 % slower: the step is bound by V, not by that load).
#include <cuda_bf16.h>

#include "hydra_internal.h"
#include "sm100_ptx.cuh"

// Compiled once per supported q / k head dimension, like the other tensor-core kernel files.
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
constexpr int kThreads = 384;
constexpr int kSlots = 2;
constexpr int kWarpProd = 8, kWarpMma = 10;            // + slot
constexpr int KV = FWD_SHORT_KEYS;                     // keys per step
constexpr uint32_t kBox = 128 * 128;                  // [128 rows x 64 bf16] = 16 KB
constexpr uint32_t kHalfBox = 64 * 128;               // [ 64 rows x 64 bf16] =  8 KB
constexpr uint32_t kQTile = kQkBoxes * kBox;
constexpr uint32_t kKStage = kQkBoxes * kHalfBox;
constexpr uint32_t kVStage = 2 * kHalfBox;
// at d_qk = 192 two slots of Q (48 KB) + two K stages (24 KB each) + one V stage (16 KB) fill the SM's shared
// memory; the S product runs two steps ahead, so K needs two stages, while V(j + 1) is only needed one
// softmax after P V(j) has released the stage
constexpr int kKStages = kDqk == 192 ? 2 : 3;
constexpr int kVStages = kDqk == 192 ? 1 : 2;
constexpr uint32_t kOffK = kQTile;
constexpr uint32_t kOffV = kOffK + kKStages * kKStage;
constexpr uint32_t kSlotBytes = kOffV + kVStages * kVStage;      // 114,688 B in both builds
constexpr uint32_t kSmemTotal = kSlots * kSlotBytes;
constexpr uint32_t kTmSlot = 256, kTmS = 128, kTmCols = 512;
constexpr float kRescaleThreshold = 8.f;              // log2 units
constexpr int kSched = 4;                             // depth of a slot's ring of work items

enum : int {
    B_QFULL = 0, B_QEMPTY = 1, B_KFULL = 2, B_KEMPTY = 5, B_VFULL = 8, B_VEMPTY = 10, B_SFULL = 12, B_PFULL = 14,
    B_PVDONE = 16, B_OFREE = 17, B_ITEMFULL = 18, B_ITEMEMPTY = 18 + kSched, B_PER_SLOT = 18 + 2 * kSched
};

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

}  // namespace

size_t HYDRA_K(fwd_short_smem_bytes)() { return kSmemTotal + 1024; }

__global__ void __launch_bounds__(kThreads, 1)
HYDRA_K(hydra_fwd_short_kernel)(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                                const __grid_constant__ CUtensorMap map_v, const FwdParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t bars[kSlots * B_PER_SLOT];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ int32_t s_sched[kSlots][kSched];
    __shared__ __align__(16) FwdShortItem s_item[kSlots][kSched];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = warp < 8 ? warp >> 2 : (warp & 1);
    const uint32_t smem = smem0 + static_cast<uint32_t>(slot) * kSlotBytes;
    const uint32_t bar0 = smem_u32(&bars[0]) + 8u * static_cast<uint32_t>(slot * B_PER_SLOT);
    auto bar = [&](int i) -> uint32_t { return bar0 + 8u * static_cast<uint32_t>(i); };

    if (tid == 0) {
        abort_flag = 0;
        const uint32_t base = smem_u32(&bars[0]);
        for (int s = 0; s < kSlots; ++s)
            for (int i = 0; i < B_PER_SLOT; ++i) {
                uint32_t count = 1u;
                if ((i >= B_PFULL && i < B_PFULL + 2) || i == B_OFREE) count = 4u;        // the slot's softmax warps
                if (i >= B_ITEMEMPTY && i < B_ITEMEMPTY + kSched) count = 5u;             // + its issuer
                mbar_init(base + 8u * static_cast<uint32_t>(s * B_PER_SLOT + i), count);
            }
        fence_mbar_init();
        tma_prefetch_desc(&map_q); tma_prefetch_desc(&map_k); tma_prefetch_desc(&map_v);
    }
    if (warp == kWarpMma) { tmem_alloc(smem_u32(&tmem_base_slot), kTmCols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_base_slot + static_cast<uint32_t>(slot) * kTmSlot;
    const uint64_t limit = p.wait_limit_ns;
    volatile int* abort_p = &abort_flag;
    auto wait = [&](int b, uint32_t parity) -> bool { return mbar_wait(bar(b), parity & 1u, abort_p, limit); };
    volatile int32_t* sched = s_sched[slot];

    if (warp == kWarpProd + slot) {
        // ------------------------------------------------------------------ work queue + TMA producer
        if (lane == 0) {
            uint32_t gk = 0, gv = 0, q_use = 0;
            bool ok = true;
            ClockProbe probe;
            probe.start();
            // test hook: idle, then hand out and load nothing; every other role's wait then runs out
            if (p.debug_stall_ns) { debug_stall(p.debug_stall_ns); ok = false; }
            int32_t* counter = &p.status->next_item[QUEUE_FWD_SHORT];
            auto fetch = [&](int raw, FwdShortItem& it) -> int {
                const int idx = raw < p.n_short ? raw : -1;
                if (idx >= 0) it = p.short_items[idx];
                return idx;
            };
            auto publish = [&](uint32_t k, int idx, const FwdShortItem& it) {
                const int rs = k % kSched;
                ok = wait(B_ITEMEMPTY + rs, (k / kSched) ^ 1u);
                if (!ok) return;
                if (idx >= 0) s_item[slot][rs] = it;
                sched[rs] = idx;
                mbar_arrive(bar(B_ITEMFULL + rs));
            };
            auto load_q = [&](const FwdShortItem& it) {
                if (!ok) return;
                ok = wait(B_QEMPTY, q_use ^ 1u);
                if (!ok) return;
                ++q_use;
                mbar_arrive_expect_tx(bar(B_QFULL), kQTile);
                for (int c = 0; c < kQkBoxes; ++c)
                    tma_load_3d(smem + c * kBox, &map_q, bar(B_QFULL), c * 64, it.head, it.q_tok0);
            };
            auto load_k = [&](const FwdShortItem& it, int j) {
                if (!ok) return;
                const int st = gk % kKStages;
                ok = wait(B_KEMPTY + st, (gk / kKStages) ^ 1u);
                if (!ok) return;
                ++gk;
                mbar_arrive_expect_tx(bar(B_KFULL + st), kKStage);
                for (int c = 0; c < kQkBoxes; ++c)
                    tma_load_3d(smem + kOffK + st * kKStage + c * kHalfBox, &map_k, bar(B_KFULL + st), c * 64,
                                it.head / p.kv_group, it.k_tok0 + j * KV);
            };
            auto load_v = [&](const FwdShortItem& it, int j) {
                if (!ok) return;
                const int st = gv % kVStages;
                ok = wait(B_VEMPTY + st, (gv / kVStages) ^ 1u);
                if (!ok) return;
                ++gv;
                mbar_arrive_expect_tx(bar(B_VFULL + st), kVStage);
                for (int c = 0; c < 2; ++c)
                    tma_load_3d(smem + kOffV + st * kVStage + c * kHalfBox, &map_v, bar(B_VFULL + st), c * 64,
                                it.head / p.kv_group, it.k_tok0 + j * KV);
            };
            // The queue is popped two items ahead and the item's descriptor one item ahead, so that neither
            // the round trip to the counter nor the load of the descriptor is ever waited for: both answers
            // are looked at one work item after they were asked for.
            FwdShortItem cur, nxt;
            int cur_idx = -1, raw1 = 0;
            if (ok) {
                const int raw0 = atomicAdd(counter, 1);
                raw1 = atomicAdd(counter, 1);
                cur_idx = fetch(raw0, cur);
                publish(0, cur_idx, cur);
            }
            bool pre = false;                          // Q and the first K tile of `cur` have been requested
            for (uint32_t kq = 0; ok && cur_idx >= 0; ++kq) {
                const int nxt_idx = fetch(raw1, nxt);
                const int raw2 = nxt_idx >= 0 ? atomicAdd(counter, 1) : 0x7fffffff;
                const int n = cur.n_kv;
                const bool nxt_loads = nxt_idx >= 0 && nxt.n_kv > 0;
                bool handed = false;                   // the next item is in the ring
                bool pre_next = false;
                auto hand_over = [&]() {
                    if (nxt_loads) { load_q(nxt); load_k(nxt, 0); pre_next = true; }
                    if (ok) publish(kq + 1, nxt_idx, nxt);
                    handed = true;
                };
                if (n > 0) {
                    if (!pre) { load_q(cur); load_k(cur, 0); }
                    if (n > 1) load_k(cur, 1);
                    for (int j = 0; j < n && ok; ++j) {
                        // The next item's Q and first K tile are released by score products that are long issued
                        // when the last V stage comes free: ask for them first, and show the item to the issuer.
                        if (j == n - 1 && n >= 2) hand_over();
                        if (j + 2 < n) load_k(cur, j + 2);       // its stage came free before V's: S(j) precedes P V(j - 1)
                        load_v(cur, j);
                    }
                }
                if (!handed && ok) hand_over();
                cur = nxt;
                cur_idx = nxt_idx;
                raw1 = raw2;
                pre = pre_next;
            }
            if (blockIdx.x == 0 && slot == 0) probe.stop(p.status, QUEUE_FWD_SHORT);
        }
    } else if (warp == kWarpMma + slot) {
        // ------------------------------------------------------------------ UMMA issuer
        if (elect_one()) {
            constexpr uint32_t idesc_s = umma_idesc_bf16(TILE, KV, false, false);
            constexpr uint32_t idesc_o = umma_idesc_bf16(TILE, D_V, false, true);
            constexpr uint32_t hi_k = umma_desc_hi(16, 1024);           // K-major Q and K boxes
            constexpr uint32_t hi_v = umma_desc_hi(kHalfBox, 1024);     // MN-major V (two 64-column boxes)
            const uint32_t q_lo = umma_desc_lo(smem, 16);
            const uint32_t k_lo0 = umma_desc_lo(smem + kOffK, 16);
            const uint32_t v_lo0 = umma_desc_lo(smem + kOffV, kHalfBox);
            // The steps of all work items of the slot form one stream, numbered gs (score products issued)
            // and gp (P V products issued). The score product runs up to two steps ahead: S(x + 1) and S(x + 2)
            // may enter the tensor pipe before P V(x), into the buffer that P V(x - 1) resp. P V(x) has read
            // (the pipe runs in issue order).
            uint32_t k_rd = 0, gs = 0, gp = 0, jobs_s = 0, jobs_p = 0;
            uint64_t fifo = 0;                         // steps of the (at most three) work items between the two
            uint32_t f_count = 0;                      // cursors, 16 bits each
            int n_s = 0, j_s = 0, n_p = 0, j_p = 0;
            bool s_have = false, s_done = false, p_have = false, ok = true;
            // One score product, if there is one to issue and (unless `blocking`) its operands have landed.
            auto issue_s = [&](bool blocking) -> bool {
                while (!s_have) {
                    if (s_done) return false;
                    const int rs = k_rd % kSched;
                    const uint32_t par = (k_rd / kSched) & 1u;
                    if (!blocking && !mbar_test_wait(bar(B_ITEMFULL + rs), par)) return false;
                    if (!wait(B_ITEMFULL + rs, par)) { ok = false; return false; }
                    const int idx = sched[rs];
                    const int n = idx >= 0 ? s_item[slot][rs].n_kv : 0;
                    mbar_arrive(bar(B_ITEMEMPTY + rs));
                    ++k_rd;
                    if (idx < 0) { s_done = true; return false; }
                    if (n <= 0) continue;
                    n_s = n; j_s = 0; s_have = true;
                    fifo |= static_cast<uint64_t>(n) << (16u * f_count);
                    ++f_count;
                }
                const uint32_t kst = gs % kKStages, kpar = (gs / kKStages) & 1u;
                if (!blocking) {
                    if (j_s == 0 && !mbar_test_wait(bar(B_QFULL), jobs_s & 1u)) return false;
                    if (!mbar_test_wait(bar(B_KFULL + kst), kpar)) return false;
                }
                if (j_s == 0 && !wait(B_QFULL, jobs_s)) { ok = false; return false; }
                if (!wait(B_KFULL + kst, kpar)) { ok = false; return false; }
                tc_fence_after_sync();
                const uint32_t d_s = tm + kTmS + (gs & 1u) * KV;
                const uint32_t b_lo = k_lo0 + kst * (kKStage >> 4);
#pragma unroll
                for (int kk = 0; kk < kDqk / 16; ++kk)
                    umma_ss_w(d_s, q_lo + (kk >> 2) * (kBox >> 4) + (kk & 3) * 2, hi_k,
                              b_lo + (kk >> 2) * (kHalfBox >> 4) + (kk & 3) * 2, hi_k, idesc_s, kk != 0);
                umma_commit(bar(B_KEMPTY + kst));
                umma_commit(bar(B_SFULL + (gs & 1u)));
                ++j_s;
                ++gs;
                if (j_s == n_s) {                      // the Q tile has had its last reader
                    umma_commit(bar(B_QEMPTY));
                    s_have = false;
                    ++jobs_s;
                }
                return true;
            };
            while (ok) {
                // P(gp) only comes once S(gp) has been computed
                while (ok && gs <= gp)
                    if (!issue_s(true)) break;
                if (!ok || gs <= gp) break;            // nothing left (or a wait ran out)
                if (gs == gp + 1u) issue_s(false);
                if (!ok) break;
                if (!p_have) {
                    n_p = static_cast<int>(fifo & 0xffffu);
                    fifo >>= 16;
                    --f_count;
                    j_p = 0;
                    p_have = true;
                }
                const uint32_t vst = gp % kVStages, vpar = (gp / kVStages) & 1u;
                ok = wait(B_VFULL + vst, vpar);
                if (ok && j_p == 0 && jobs_p > 0) ok = wait(B_OFREE, jobs_p - 1u);   // the previous item's O is out
                if (ok) ok = wait(B_PFULL + (gp & 1u), gp >> 1);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t a_p = tm + kTmS + (gp & 1u) * KV;
                const uint32_t b_lo = v_lo0 + vst * (kVStage >> 4);
#pragma unroll
                for (int kk = 0; kk < KV / 16; ++kk)
                    umma_ts_w(tm, a_p + kk * 8, b_lo + kk * (2048 >> 4), hi_v, idesc_o, (j_p | kk) != 0);
                umma_commit(bar(B_VEMPTY + vst));
                umma_commit(bar(B_PVDONE));
                ++j_p;
                ++gp;
                if (j_p == n_p) { p_have = false; ++jobs_p; }
            }
        }
    } else if (warp < 8) {
        // ------------------------------------------------------------------ softmax warps
        const int r = tid & 127;                       // row of the tile = TMEM lane
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tm_o = tm + lane_base;
        const uint32_t tm_s0 = tm + kTmS + lane_base;
        uint32_t g = 0;                                // steps of this slot so far
        bool ok = true;
        for (uint32_t kq = 0; ok; ++kq) {
            const int rs = kq % kSched;
            ok = wait(B_ITEMFULL + rs, kq / kSched);
            if (!ok) break;
            const int idx = sched[rs];
            FwdShortItem item;
            if (idx >= 0) item = s_item[slot][rs];
            mbar_arrive_warp(bar(B_ITEMEMPTY + rs));
            if (idx < 0) break;
            const bool row_valid = r < item.rows;
            const int64_t rows_total = item.to_part ? p.part_rows : p.T;
            __nv_bfloat16* obase = static_cast<__nv_bfloat16*>(item.to_part ? p.o_part : p.out);
            float* lbase = item.to_part ? p.lse_part : p.lse;
            const int64_t orow = static_cast<int64_t>(item.out_row0) + r;
            uint4* dst = reinterpret_cast<uint4*>(obase + (orow * p.h + item.head) * D_V);
            float* lse_dst = lbase + static_cast<int64_t>(item.head) * rows_total + orow;
            const int n_kv = item.n_kv;
            if (n_kv <= 0) {                           // rows that see no key: O = 0, LSE = -inf
                if (row_valid) {
#pragma unroll
                    for (int e = 0; e < D_V / 8; ++e) dst[e] = make_uint4(0u, 0u, 0u, 0u);
                    *lse_dst = neg_inf();
                }
                continue;
            }
            float m_run = neg_inf(), l_run = 0.f;
            for (int j = 0; j < n_kv && ok; ++j, ++g) {
                const uint32_t b = g & 1u;
                ok = wait(B_SFULL + b, g >> 1);
                if (!ok) break;
                tc_fence_after_sync();
                const int col0 = j * KV;
                // key col0 + c is visible to row r iff it exists and (causal) c0 + c <= r + off
                const bool need_mask = (col0 + KV > item.k_len) || (p.causal && (col0 + KV - 1 > item.off));
                int cmax = KV;                         // columns 0..cmax are visible
                if (need_mask) {
                    int jmax = item.k_len - 1;
                    if (p.causal) jmax = min(jmax, r + item.off);
                    cmax = jmax - col0;
                }
                uint32_t s[KV];
                tmem_ld_x32(tm_s0 + b * KV, s);
                tmem_ld_x32(tm_s0 + b * KV + 32, s + 32);
                tmem_wait_ld();
                if (need_mask) {
#pragma unroll
                    for (int c = 0; c < KV; ++c)
                        if (c > cmax) s[c] = __float_as_uint(neg_inf());
                }
                float mx0 = neg_inf(), mx1 = neg_inf(), mx2 = neg_inf(), mx3 = neg_inf();
#pragma unroll
                for (int c = 0; c < KV; c += 8) {
                    mx0 = fmax3(mx0, __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
                    mx1 = fmax3(mx1, __uint_as_float(s[c + 2]), __uint_as_float(s[c + 3]));
                    mx2 = fmax3(mx2, __uint_as_float(s[c + 4]), __uint_as_float(s[c + 5]));
                    mx3 = fmax3(mx3, __uint_as_float(s[c + 6]), __uint_as_float(s[c + 7]));
                }
                const float m_new = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2;
                float alpha = 1.f;
                if (m_new > m_run + kRescaleThreshold || (j == 0)) {
                    alpha = ex2_approx(m_run - m_new);          // 0 when m_run = -inf
                    if (m_new == neg_inf()) alpha = 1.f;         // nothing visible yet: keep -inf
                    else m_run = m_new;
                }
                const float m_use = (m_run == neg_inf()) ? 0.f : m_run;
                // masked scores are -inf in registers since the maximum was taken, so their probabilities come out
                // as exp2(-inf) = 0 by themselves: one code path for interior and diagonal steps
                uint32_t pk[KV / 2];
                float rs0 = 0.f, rs1 = 0.f;
#pragma unroll
                for (int c = 0; c < KV; c += 2) {
                    float x0, x1;
                    ffma2(x0, x1, __uint_as_float(s[c]), __uint_as_float(s[c + 1]), p.scale_log2, p.scale_log2,
                          -m_use, -m_use);
                    const float p0 = ex2_approx(x0);
                    const float p1 = ex2_approx(x1);
                    fadd2(rs0, rs1, rs0, rs1, p0, p1);
                    pk[c >> 1] = pack_bf16x2(p0, p1);
                }
                // Every thread looks at every phase of "P V done" exactly once (a phase skipped could not be told
                // from the one after next), here, where the previous product has long completed; O is rescaled
                // after the exponentials so that the scores need not stay in registers next to it.
                if (j > 0) {
                    ok = wait(B_PVDONE, g - 1u);
                    if (!ok) break;
                    if (__any_sync(0xffffffffu, alpha != 1.f)) {
                        tc_fence_after_sync();
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
                }
                tmem_st_x32(tm_s0 + b * KV, pk);
                tmem_wait_st();
                tc_fence_before_sync();
                mbar_arrive_warp(bar(B_PFULL + b));
                l_run = l_run * alpha + (rs0 + rs1);
            }
            if (!ok) break;
            // ---- epilogue: O / l -> bf16, LSE = ln2 * (m + log2 l) ---------------------------------
            ok = wait(B_PVDONE, g - 1u);
            if (!ok) break;
            tc_fence_after_sync();
            const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
            const bool wide = (reinterpret_cast<uintptr_t>(dst) & 31u) == 0;   // the interface asks for 16 bytes only
#pragma unroll
            for (int c0 = 0; c0 < D_V; c0 += 32) {
                uint32_t o[32];
                tmem_ld_x32(tm_o + c0, o);
                tmem_wait_ld();
                if (c0 + 32 == D_V) {                  // every column has left TMEM: O may be overwritten
                    tc_fence_before_sync();
                    mbar_arrive_warp(bar(B_OFREE));
                }
                if (row_valid) {
                    // 32 bytes per store: a thread's row is 4 KB away from its neighbour's, so every store of the
                    // warp touches 32 lines; whole sectors halve the number of such instructions
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
    if (warp == kWarpMma) tmem_dealloc(tmem_base_slot, kTmCols);
}

cudaError_t HYDRA_K(launch_fwd_short)(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                                      const FwdParams& p, int grid, cudaStream_t stream)
{
    // the opt-in to more than 48 KB of dynamic shared memory is made once per device ordinal
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        e = cudaFuncSetAttribute(HYDRA_K(hydra_fwd_short_kernel), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(HYDRA_K(fwd_short_smem_bytes)()));
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    HYDRA_K(hydra_fwd_short_kernel)<<<grid, kThreads, HYDRA_K(fwd_short_smem_bytes)(), stream>>>(mq, mk, mv, p);
    return cudaGetLastError();
}

}  // namespace hydra
