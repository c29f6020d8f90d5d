// Backward attention on sm_100a, as two kernels whose accumulators never leave the chip:
//   hydra_bwd_dq_kernel   q-stationary: one 128-row q tile visits every kv tile of every pair of its
//                         q chunk; dQ (128 x 192 fp32) stays in tensor memory and is written once.
//   hydra_bwd_dkv_kernel  kv-stationary: one 128-row kv tile visits, in 64-row q sub-tiles, every
//                         pair of its kv chunk; dK (128 x 192) and dV (128 x 128) stay in tensor
//                         memory and are written once.
// Both recompute S and dP = dO V^T from the inputs, form P = exp2(S*c - LSE*log2e) and
// dS = P (dP - D) on thread-private rows, hand P / dS back to the tensor core as packed bf16 in
// tensor memory (A operand of a TS UMMA), and read Q / K / dO as MN-major B operands straight from
// their token-major TMA tiles, so nothing is transposed in shared memory.
//
// Warp roles (352 threads) in both kernels:
//   warps 0-3, 4-7  two elementwise warpgroups; thread r of each owns tile row r = TMEM lane r and
//                   one half of the columns of S / dP
//   warp 8          TMA producer (plus the LSE / D loads of the dK/dV kernel)
//   warp 9          UMMA issuer of the score products (S, dP); owner of the TMEM allocation
//   warp 10         UMMA issuer of the gradient updates (dQ, or dV and dK)
// The elementwise threads copy S and dP to registers and release them at once, so that the UMMAs of
// the next step run while the exponentials of this one are computed.
#include <cuda_bf16.h>

#include "hydra_internal.h"
#include "sm100_ptx.cuh"

// This file is compiled once per supported q / k head dimension (HYDRA_KERNEL_DQK = 192, the default, or
// 128); the value dimension is 128 in both. HYDRA_K() gives the kernels and launchers of the second
// build their own names. The tensor-memory maps are those of d_qk = 192 in both builds (at 128 a third of
// the dQ / dK columns stays unused).
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
constexpr int kQkBoxes = kDqk / 64;        // 64-column boxes of a q / k row
constexpr int kThreads = 352;
constexpr int kWarpProd = 8, kWarpMma = 9, kWarpMma2 = 10;
constexpr uint32_t kBox128 = 128 * 128;   // [128 rows x 64 bf16]
constexpr uint32_t kBox64 = 64 * 128;     // [ 64 rows x 64 bf16]
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kSched = 4;                  // depth of the in-CTA ring of work-item indices

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }
__device__ __forceinline__ float pos_inf() { return __int_as_float(0x7f800000); }

// n (a multiple of 16) values of a thread's own row. Rows of neighbouring threads are kilobytes apart, so every
// store of the warp touches 32 lines: 32-byte stores (one sector per thread) where the address allows it (the
// interface asks for 16-byte alignment only) halve the number of such instructions.
__device__ __forceinline__ void store_row_bf16(__nv_bfloat16* dst, const uint32_t* v, int n, float mul)
{
    uint4* d4 = reinterpret_cast<uint4*>(dst);
    const bool wide = (reinterpret_cast<uintptr_t>(dst) & 31u) == 0;
#pragma unroll
    for (int e = 0; e < n; e += 16) {
        uint32_t w[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
            w[i] = pack_bf16x2(__uint_as_float(v[e + 2 * i]) * mul, __uint_as_float(v[e + 2 * i + 1]) * mul);
        if (wide) {
            st_global_v8(d4 + (e >> 3), w);
        } else {
            d4[e >> 3] = make_uint4(w[0], w[1], w[2], w[3]);
            d4[(e >> 3) + 1] = make_uint4(w[4], w[5], w[6], w[7]);
        }
    }
}

// Warp-cooperative form of store_row_bf16 for an epilogue that nothing overlaps: lane l holds 32 values
// of row l of the warp's 32 rows (rows `row_stride` elements apart in memory). Written straight from
// registers, every store instruction would touch 32 cache lines (16 bytes in each) and the 20 of them an
// epilogue needs keep the load/store unit busy for thousands of cycles; transposed through a 2 KB slice
// of shared memory, lane l stores chunk l % 4 of rows l / 4 + 8 e: eight 64-byte segments per instruction.
// `dst` is this lane's own row pointer, `valid` the ballot of the rows that exist.
__device__ __forceinline__ void store_rows_bf16_coalesced(uint32_t slice, int lane, __nv_bfloat16* dst,
                                                          int64_t row_stride, const uint32_t* v, float mul, uint32_t valid)
{
    __syncwarp();                                      // earlier reads of the slice are over
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const uint32_t w0 = pack_bf16x2(__uint_as_float(v[8 * e + 0]) * mul, __uint_as_float(v[8 * e + 1]) * mul);
        const uint32_t w1 = pack_bf16x2(__uint_as_float(v[8 * e + 2]) * mul, __uint_as_float(v[8 * e + 3]) * mul);
        const uint32_t w2 = pack_bf16x2(__uint_as_float(v[8 * e + 4]) * mul, __uint_as_float(v[8 * e + 5]) * mul);
        const uint32_t w3 = pack_bf16x2(__uint_as_float(v[8 * e + 6]) * mul, __uint_as_float(v[8 * e + 7]) * mul);
        st_shared_v4(slice + lane * 64 + ((e ^ ((lane >> 1) & 3)) << 4), w0, w1, w2, w3);
    }
    __syncwarp();
    __nv_bfloat16* base = dst - static_cast<int64_t>(lane) * row_stride + (lane & 3) * 8;   // row 0 of the warp, this lane's chunk
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int row = 8 * e + (lane >> 2);
        const uint4 w = ld_shared_v4(slice + row * 64 + (((lane & 3) ^ ((row >> 1) & 3)) << 4));
        if ((valid >> row) & 1u) *reinterpret_cast<uint4*>(base + row * row_stride) = w;
    }
}

// The accumulating counterpart: 16 fp32 columns (64 bytes per row) per call through the same slice, then
// 16-byte reductions of whole 64-byte row segments.
__device__ __forceinline__ void add_rows_f32_coalesced(uint32_t slice, int lane, float* dst, int64_t row_stride,
                                                       const uint32_t* v, float mul, uint32_t valid)
{
    __syncwarp();
#pragma unroll
    for (int e = 0; e < 4; ++e)
        st_shared_v4(slice + lane * 64 + ((e ^ ((lane >> 1) & 3)) << 4), __float_as_uint(__uint_as_float(v[4 * e + 0]) * mul),
                     __float_as_uint(__uint_as_float(v[4 * e + 1]) * mul), __float_as_uint(__uint_as_float(v[4 * e + 2]) * mul),
                     __float_as_uint(__uint_as_float(v[4 * e + 3]) * mul));
    __syncwarp();
    float* base = dst - static_cast<int64_t>(lane) * row_stride + (lane & 3) * 4;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int row = 8 * e + (lane >> 2);
        const uint4 w = ld_shared_v4(slice + row * 64 + (((lane & 3) ^ ((row >> 1) & 3)) << 4));
        if ((valid >> row) & 1u)
            red_add_v4_f32(base + row * row_stride, __uint_as_float(w.x), __uint_as_float(w.y), __uint_as_float(w.z),
                           __uint_as_float(w.w));
    }
}

// Accumulating form of the same epilogue: dst (fp32) += v * mul, as 16-byte reductions performed at
// the L2 cache. Every row is owned by one thread of one CTA per launch and launches on a stream are
// ordered, so every address receives one addition per launch and the sum does not depend on timing;
// a reduction is used instead of load-add-store only because it does not make the thread wait for
// the old value (five dependent round trips to memory per work item otherwise).
__device__ __forceinline__ void add_row_f32(float* dst, const uint32_t* v, int n, float mul)
{
#pragma unroll
    for (int e = 0; e < n; e += 4)
        red_add_v4_f32(dst + e, __uint_as_float(v[e + 0]) * mul, __uint_as_float(v[e + 1]) * mul,
                       __uint_as_float(v[e + 2]) * mul, __uint_as_float(v[e + 3]) * mul);
}

// ---------------------------------------------------------------------------------------------
// dQ kernel: layout
// ---------------------------------------------------------------------------------------------
namespace dq {
constexpr int kKStages = 2, kVSlots = 3;
constexpr uint32_t kQ = 0;                                   // kQkBoxes boxes of 64 columns, stationary
constexpr uint32_t kDO = kQ + kQkBoxes * kBox128;                   // 2 boxes, stationary
constexpr uint32_t kK = kDO + 2 * kBox128;                   // 2 stages x kQkBoxes boxes
constexpr uint32_t kV = kK + kKStages * kQkBoxes * kBox128;         // ring of 3 boxes [128 kv x 64 d_v]
constexpr uint32_t kTotal = kV + kVSlots * kBox128;          // 229,376 B at d_qk = 192
constexpr uint32_t kTmS = 0, kTmDP = 128, kTmDQ = 256, kTmDS = 448, kTmCols = 512;
// K-full is kept per 64-column box (3 per stage): S = Q K^T consumes the boxes in order, so it starts
// when the first 16 KB have landed instead of waiting for all 48 KB of the stage.
enum : int { B_QFULL = 0, B_QEMPTY = 1, B_KFULL = 2, B_KEMPTY = 8, B_VFULL = 10, B_VEMPTY = 13,
             B_SFULL = 16, B_SFREE = 17, B_PFULL = 18, B_DSFREE = 20, B_ACCFREE = 21, B_DPFULL = 22, B_DPFREE = 23,
             B_ITEMFULL = 24, B_ITEMEMPTY = 24 + kSched, B_COUNT = 24 + 2 * kSched };

// Iterator over (pair of the q chunk, kv tile) in the order every role walks them.
struct TileIter {
    const PairDev* pairs; const int32_t* list; int list_len; int last_row; int causal;
    int li, t, nt; PairDev cur;
    __device__ int tiles_of(const PairDev& pr) const {
        int n_keys = pr.k_len;
        if (causal) n_keys = min(n_keys, last_row + pr.off + 1);
        return n_keys > 0 ? (n_keys + TILE - 1) / TILE : 0;
    }
    __device__ void seek() {
        while (li < list_len) {
            if (li > 0) cur = pairs[list[li]];
            nt = tiles_of(cur);
            if (nt > 0) return;
            ++li;
        }
    }
    // `first` = pairs[list[0]], which the caller already holds (from the work ring in shared memory)
    __device__ void init(const PairDev* p, const int32_t* l, int n, int lr, int c, const PairDev& first) {
        pairs = p; list = l; list_len = n; last_row = lr; causal = c; li = 0; t = 0; nt = 0; cur = first;
        seek();
    }
    __device__ bool valid() const { return li < list_len; }
    __device__ void next() { if (++t >= nt) { t = 0; ++li; seek(); } }
};
}  // namespace dq

// ---------------------------------------------------------------------------------------------
// dK/dV kernel: layout
// ---------------------------------------------------------------------------------------------
namespace dkv {
constexpr int kStages = 3;
constexpr uint32_t kK = 0;                                   // kQkBoxes boxes of 128 rows, stationary
constexpr uint32_t kV = kK + kQkBoxes * kBox128;                    // 2 boxes of 128 rows, stationary
constexpr uint32_t kQ = kV + 2 * kBox128;                    // stages x kQkBoxes boxes of 64 rows
constexpr uint32_t kDO = kQ + kStages * kQkBoxes * kBox64;          // stages x 2 boxes of 64 rows
constexpr uint32_t kDsStage = kDO + kStages * 2 * kBox64;    // 8 warps x 2 KB: dK / dV rows on their way to memory
constexpr uint32_t kTotal = kDsStage + 8 * 2048;             // 221,184 B at d_qk = 192
constexpr uint32_t kTmDK = 0, kTmDV = 192, kTmS = 320, kTmDP = 384, kTmP = 448, kTmDS = 480,
                   kTmCols = 512;
enum : int { B_KVFULL = 0, B_KVEMPTY = 1, B_QFULL = 2, B_STAT = 5, B_QEMPTY = 8, B_SFULL = 11,
             B_SFREE = 12, B_PFULL = 13, B_PDSFREE = 14, B_ACCFREE = 15, B_ITEMFULL = 16, B_ITEMEMPTY = 16 + kSched,
             B_COUNT = 16 + 2 * kSched };

// Iterator over (pair of the kv chunk, 64-row q sub-tile).
struct SubIter {
    const PairDev* pairs; const int32_t* list; int list_len; int r0; int causal; int even;
    int li, u, nu; PairDev cur;
    __device__ void seek() {
        while (li < list_len) {
            if (li > 0) cur = pairs[list[li]];
            nu = (cur.q_len + SUB - 1) / SUB;
            u = 0;
            if (causal) { const int i_min = r0 - cur.off; u = i_min > 0 ? i_min / SUB : 0; }
            // with the dS hand-off a q tile is read as two sub-tiles: start at the even one (the extra
            // sub-tile, if any, is fully masked and contributes zeros)
            if (even) u &= ~1;
            if (u < nu) return;
            ++li;
        }
    }
    __device__ void init(const PairDev* p, const int32_t* l, int n, int r, int c, int ev, const PairDev& first) {
        pairs = p; list = l; list_len = n; r0 = r; causal = c; even = ev; li = 0; u = 0; nu = 0; cur = first;
        seek();
    }
    __device__ bool valid() const { return li < list_len; }
    __device__ void next() { if (++u >= nu) { ++li; seek(); } }
};
}  // namespace dkv

}  // namespace

size_t HYDRA_K(bwd_dq_smem_bytes)() { return dq::kTotal + 1024; }
size_t HYDRA_K(bwd_dkv_smem_bytes)() { return dkv::kTotal + 1024; }

// =============================================================================================
// dQ
// =============================================================================================
__global__ void __launch_bounds__(kThreads, 1)
HYDRA_K(hydra_bwd_dq_kernel)(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do,
                    const BwdParams p)
{
    using namespace dq;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem = (smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t bars[B_COUNT];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ int32_t s_sched[kSched];
    __shared__ GroupItem s_item[kSched];              // the work ring carries the item and its first pair, so that
    __shared__ PairDev s_first[kSched];               // no role starts an item with a walk through global memory

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t bar0 = smem_u32(&bars[0]);
    auto bar = [&](int i) -> uint32_t { return bar0 + 8u * static_cast<uint32_t>(i); };
    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < B_COUNT; ++i) {
            const bool by_threads = (i == B_SFREE) || (i == B_DPFREE) || (i == B_PFULL) || (i == B_PFULL + 1) ||
                                    (i == B_ACCFREE);
            const bool by_readers = i >= B_ITEMEMPTY && i < B_ITEMEMPTY + kSched;
            mbar_init(bar(i), by_readers ? 10u : (by_threads ? 8u : 1u));   // 8 elementwise warps (+ 2 issuers)
        }
        fence_mbar_init();
        tma_prefetch_desc(&map_q); tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v); tma_prefetch_desc(&map_do);
    }
    if (warp == kWarpMma) { tmem_alloc(smem_u32(&tmem_base_slot), kTmCols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_base_slot;
    const uint64_t limit = p.wait_limit_ns;
    volatile int* abort_p = &abort_flag;
    auto wait = [&](int b, uint32_t parity) -> bool { return mbar_wait(bar(b), parity & 1u, abort_p, limit); };
    // Work queue: the producer pops the next item index from a counter in global memory (so a CTA that
    // finishes early simply takes more items: no cost model has to predict the run time of an item)
    // and hands it to the other warps of the CTA through a small ring in shared memory.
    volatile int32_t* sched = s_sched;
    // The pop is split in two: the request to the counter goes out when an item starts, its answer is
    // looked at after the first loads of that item have been issued; the producer then fetches the
    // next item's descriptors (three dependent loads from global memory) and puts them in the ring.
    constexpr int kPopFailed = 0x7fffffff;
    auto pop_begin = [&](uint32_t k) -> int {               // producer, one thread
        const int slot = k % kSched;
        if (!mbar_wait(bar(B_ITEMEMPTY + slot), ((k / kSched) ^ 1u) & 1u, abort_p, limit)) return kPopFailed;
        return atomicAdd(&p.status->next_item[QUEUE_DQ], 1);
    };
    auto pop_end = [&](uint32_t k, int raw, GroupItem& item_out, PairDev& first_out) -> int {
        if (raw == kPopFailed) return -1;
        const int slot = k % kSched;
        const int idx = raw >= p.n_items ? -1 : raw;
        if (idx >= 0) {
            item_out = p.items[idx];
            first_out = p.pairs[p.lists[item_out.list_off]];
            s_item[slot] = item_out;
            s_first[slot] = first_out;
        }
        sched[slot] = idx;
        mbar_arrive(bar(B_ITEMFULL + slot));
        return idx;
    };
    auto next_item = [&](uint32_t k, GroupItem& item_out, PairDev& first_out) -> int {   // every other warp, all lanes
        const int slot = k % kSched;
        if (!mbar_wait(bar(B_ITEMFULL + slot), (k / kSched) & 1u, abort_p, limit)) return -1;
        const int idx = sched[slot];
        if (idx >= 0) {
            item_out = s_item[slot];
            first_out = s_first[slot];
        }
        mbar_arrive_warp(bar(B_ITEMEMPTY + slot));
        return idx;
    };

    if (warp == kWarpProd) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t items = 0, gk = 0, gv = 0;
            bool ok = true;
            ClockProbe probe;
            probe.start();
            // one item ahead: the round trip to the counter and the descriptor fetch overlap the loads of
            // the current item
            GroupItem item_next;
            PairDev first_next;
            // test hook: idle, then hand out and load nothing; every other role's wait then runs out
            if (p.debug_stall_ns) { debug_stall(p.debug_stall_ns); ok = false; }
            int it_ahead = ok ? pop_end(0, pop_begin(0), item_next, first_next) : -1;
            for (uint32_t kq = 0; ok; ++kq) {
                const int it = it_ahead;
                if (it < 0) break;
                const GroupItem item = item_next;
                const PairDev first = first_next;
                const int raw_next = pop_begin(kq + 1);
                bool popped = false;
                const int32_t* list = p.lists + item.list_off;
                TileIter ti;
                ti.init(p.pairs, list, item.list_len, min(item.r0 + TILE, first.q_len) - 1, p.causal, first);
                if (!ti.valid()) { it_ahead = pop_end(kq + 1, raw_next, item_next, first_next); continue; }
                ok = wait(B_QEMPTY, items ^ 1u);
                if (!ok) break;
                ++items;
                mbar_arrive_expect_tx(bar(B_QFULL), (kQkBoxes + 2) * kBox128);
                for (int c = 0; c < kQkBoxes; ++c)
                    tma_load_3d(smem + kQ + c * kBox128, &map_q, bar(B_QFULL), c * 64, item.head,
                                first.q_tok0 + item.r0);
                for (int c = 0; c < 2; ++c)
                    tma_load_3d(smem + kDO + c * kBox128, &map_do, bar(B_QFULL), c * 64, item.head,
                                first.q_tok0 + item.r0);
                for (; ti.valid() && ok; ti.next()) {
                    const int tok = ti.cur.k_tok0 + ti.t * TILE;
                    // V first: its slots were freed a whole tile ago and dP is the first product of the
                    // tile; the K stage frees only when the dQ update two tiles back has completed
                    for (int c = 0; c < 2 && ok; ++c, ++gv) {
                        const int slot = gv % kVSlots;
                        ok = wait(B_VEMPTY + slot, (gv / kVSlots) ^ 1u);
                        if (!ok) break;
                        mbar_arrive_expect_tx(bar(B_VFULL + slot), kBox128);
                        tma_load_3d(smem + kV + slot * kBox128, &map_v, bar(B_VFULL + slot), c * 64,
                                    item.head / p.kv_group, tok);
                    }
                    if (!ok) break;
                    const int st = gk % kKStages;
                    ok = wait(B_KEMPTY + st, (gk / kKStages) ^ 1u);
                    if (!ok) break;
                    ++gk;
                    for (int c = 0; c < kQkBoxes; ++c) {
                        mbar_arrive_expect_tx(bar(B_KFULL + st * 3 + c), kBox128);
                        tma_load_3d(smem + kK + st * kQkBoxes * kBox128 + c * kBox128, &map_k, bar(B_KFULL + st * 3 + c),
                                    c * 64, item.head / p.kv_group, tok);
                    }
                    if (!popped) { it_ahead = pop_end(kq + 1, raw_next, item_next, first_next); popped = true; }
                }
                if (!popped) it_ahead = pop_end(kq + 1, raw_next, item_next, first_next);
            }
            if (blockIdx.x == 0) probe.stop(p.status, QUEUE_DQ);
        }
    } else if (warp == kWarpMma || warp == kWarpMma2) {
        // ------------------------------------------------------------------ UMMA issuers
        // Two issuing threads, so that neither kind of UMMA waits behind the other's operands:
        // warp 9 issues S = Q K^T and dP = dO V^T of tile j+1 as soon as S/dP of tile j have been
        // copied out and K, V have landed; warp 10 issues dQ += dS K of tile j as soon as dS is there.
        // The whole warp walks the work list (uniform control flow, so addresses and descriptors stay
        // on the uniform datapath); one elected lane issues the UMMAs and commits.
        {
            constexpr uint32_t idesc_s = umma_idesc_bf16(TILE, TILE, false, false);
            constexpr uint32_t idesc_dq = umma_idesc_bf16(TILE, kDqk, false, true);
            constexpr uint32_t hi_kmaj = umma_desc_hi(16, 1024);
            constexpr uint32_t hi_kmn = umma_desc_hi(kBox128, 1024);       // K as MN-major B, N = 192
            const uint32_t q_lo = umma_desc_lo(smem + kQ, 16), do_lo = umma_desc_lo(smem + kDO, 16);
            const uint32_t k_lo0 = umma_desc_lo(smem + kK, 16), v_lo0 = umma_desc_lo(smem + kV, 16);
            const uint32_t kmn_lo0 = umma_desc_lo(smem + kK, kBox128);
            const bool issue_scores = warp == kWarpMma;
            uint32_t items = 0, n_tile = 0, gv = 0;       // running counts of this issuer
            bool ok = true;
            for (uint32_t kq = 0; ok; ++kq) {
                GroupItem item;
                PairDev first;
                const int it = next_item(kq, item, first);
                if (it < 0) break;
                const int32_t* list = p.lists + item.list_off;
                TileIter ti;
                ti.init(p.pairs, list, item.list_len, min(item.r0 + TILE, first.q_len) - 1, p.causal, first);
                if (!ti.valid()) continue;
                if (issue_scores) {
                    ok = wait(B_QFULL, items);
                    for (; ti.valid() && ok;) {
                        // dP and S are handed over separately. dP comes first (V was loaded a whole tile
                        // ago, while the K stage of this tile was freed only by the dQ update two tiles
                        // back and may still be landing); the elementwise warps copy it out while S is
                        // still being computed, so the dP of the next tile can follow this S at once and
                        // fills the time in which S is copied out.
                        if (n_tile > 0) ok = wait(B_DPFREE, n_tile - 1u);  // previous dP is in registers
                        if (!ok) break;
#pragma unroll
                        for (int c = 0; c < 2; ++c, ++gv) {
                            const int slot = gv % kVSlots;
                            ok = wait(B_VFULL + slot, gv / kVSlots);
                            if (!ok) break;
                            tc_fence_after_sync();
                            const uint32_t v_lo = v_lo0 + slot * (kBox128 >> 4);
                            if (elect_one()) {
#pragma unroll
                                for (int kk = 0; kk < 4; ++kk)
                                    umma_ss_w(tm + kTmDP, do_lo + c * (kBox128 >> 4) + kk * 2, hi_kmaj, v_lo + kk * 2,
                                              hi_kmaj, idesc_s, (c | kk) != 0);
                                umma_commit(bar(B_VEMPTY + slot));
                                if (c == 1) umma_commit(bar(B_DPFULL));
                            }
                        }
                        if (!ok) break;
                        if (n_tile > 0) ok = wait(B_SFREE, n_tile - 1u);   // previous S is in registers
                        if (!ok) break;
                        const int st = n_tile % kKStages;
                        const uint32_t k_lo = k_lo0 + st * (kQkBoxes * kBox128 >> 4);
#pragma unroll
                        for (int c = 0; c < kQkBoxes; ++c) {
                            ok = wait(B_KFULL + st * 3 + c, n_tile / kKStages);
                            if (!ok) break;
                            tc_fence_after_sync();
                            if (elect_one()) {
#pragma unroll
                                for (int kk = 0; kk < 4; ++kk) {
                                    const uint32_t o = c * (kBox128 >> 4) + kk * 2;
                                    umma_ss_w(tm + kTmS, q_lo + o, hi_kmaj, k_lo + o, hi_kmaj, idesc_s, (c | kk) != 0);
                                }
                                if (c == kQkBoxes - 1) umma_commit(bar(B_SFULL));
                            }
                        }
                        if (!ok) break;
                        ++n_tile;
                        ti.next();
                        if (!ti.valid() && elect_one()) umma_commit(bar(B_QEMPTY));     // Q and dO are no longer read
                    }
                } else {
                    bool first_tile = true;
                    for (; ti.valid() && ok; ti.next()) {
                        // dS arrives in two instalments: columns [0,32) of each half (K-steps 0,1,4,5),
                        // then columns [32,64) (K-steps 2,3,6,7); the update of the first overlaps the
                        // exponentials of the second
                        const int st = n_tile % kKStages;
                        const uint32_t k_lo = kmn_lo0 + st * (kQkBoxes * kBox128 >> 4);
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            ok = wait(B_PFULL + half, n_tile);
                            if (ok && half == 0 && first_tile && items > 0) ok = wait(B_ACCFREE, items - 1u);
                            if (!ok) break;
                            tc_fence_after_sync();
                            if (elect_one()) {
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int kk = (e >> 1) * 4 + half * 2 + (e & 1);
                                    umma_ts_w(tm + kTmDQ, tm + kTmDS + kk * 8, k_lo + kk * (2048 >> 4), hi_kmn, idesc_dq,
                                              (half > 0 || e > 0 || !first_tile) ? 1u : 0u);
                                }
                                if (half == 1) {
                                    umma_commit(bar(B_DSFREE));
                                    umma_commit(bar(B_KEMPTY + st));
                                }
                            }
                        }
                        if (!ok) break;
                        ++n_tile;
                        first_tile = false;
                    }
                }
                ++items;
            }
        }
    } else {
        // ------------------------------------------------------------------ elementwise warpgroups
        const int g = warp >> 2;                       // column half
        const int r = tid & 127;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tm_s = tm + kTmS + lane_base + g * 64;
        const uint32_t tm_dp = tm + kTmDP + lane_base + g * 64;
        const uint32_t tm_ds = tm + kTmDS + lane_base + g * 32;
        uint32_t c_s = 0, c_ds = 0;
        bool ok = true;
        for (uint32_t kq = 0; ok; ++kq) {
            GroupItem item;
            PairDev first;
            const int it = next_item(kq, item, first);
            if (it < 0) break;
            const int32_t* list = p.lists + item.list_off;
            const int row = item.r0 + r;
            const bool row_valid = row < first.q_len;
            const int64_t dst_off = (static_cast<int64_t>(first.q_tok0 + row) * p.h + item.head) * kDqk + g * (kDqk / 2);
            __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(p.dq) + dst_off;
            float* dst_acc = static_cast<float*>(p.dq) + dst_off;        // accumulate mode: dq is fp32
            TileIter ti;
            ti.init(p.pairs, list, item.list_len, min(item.r0 + TILE, first.q_len) - 1, p.causal, first);
            if (!ti.valid()) {                         // no visible key at all: dQ = 0 (nothing to add)
                if (row_valid && !p.accumulate) {
                    uint4* d4 = reinterpret_cast<uint4*>(dst);
#pragma unroll
                    for (int e = 0; e < kDqk / 16; ++e) d4[e] = make_uint4(0u, 0u, 0u, 0u);
                }
                continue;
            }
            float lse2 = 0.f, dsum = 0.f;
            if (row_valid) {
                const float l = p.lse[static_cast<int64_t>(item.head) * p.T + first.q_tok0 + row];
                lse2 = (l == neg_inf()) ? pos_inf() : l * kLog2e;
                dsum = p.dsum[static_cast<int64_t>(item.head) * p.T + first.q_tok0 + row];
            }
            for (; ti.valid() && ok; ti.next()) {
                uint32_t s[64], dp[64];
                ok = wait(B_DPFULL, c_s);
                if (!ok) break;
                tc_fence_after_sync();
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) tmem_ld_x32(tm_dp + c0, dp + c0);
                tmem_wait_ld();
                tc_fence_before_sync();
                mbar_arrive_warp(bar(B_DPFREE));            // the next dP may overwrite tensor memory
                ok = wait(B_SFULL, c_s);
                ++c_s;
                if (!ok) break;
                tc_fence_after_sync();
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) tmem_ld_x32(tm_s + c0, s + c0);
                tmem_wait_ld();
                tc_fence_before_sync();
                // the next S may overwrite tensor memory; the arrival must not sink below the arithmetic
                const float lse2_t = mbar_arrive_warp_before(bar(B_SFREE), lse2);
                int jmax = ti.cur.k_len - 1;
                if (p.causal) jmax = min(jmax, row + ti.cur.off);
                const int cmax = jmax - ti.t * TILE - g * 64;      // columns 0..cmax of this half are visible
                uint32_t ds[32];
                float lse2_h = lse2_t;
                // Interior tiles (every column visible to every row of the warp) skip the masking; elsewhere the
                // masked scores become -inf, whose probability exp2(-inf) is 0 by itself: one arithmetic path.
                if (__any_sync(0xffffffffu, cmax < 63)) {
#pragma unroll
                    for (int c = 0; c < 64; ++c)
                        if (c > cmax) s[c] = __float_as_uint(neg_inf());
                }
#pragma unroll
                for (int half = 0; half < 2; ++half) {
#pragma unroll
                    for (int c = half * 32; c < half * 32 + 32; c += 2) {
                        float x0, x1, d0, d1;
                        ffma2(x0, x1, __uint_as_float(s[c]), __uint_as_float(s[c + 1]), p.scale_log2, p.scale_log2,
                              -lse2_h, -lse2_h);
                        fadd2(d0, d1, __uint_as_float(dp[c]), __uint_as_float(dp[c + 1]), -dsum, -dsum);
                        fmul2(d0, d1, d0, d1, ex2_approx(x0), ex2_approx(x1));
                        ds[c >> 1] = pack_bf16x2(d0, d1);
                    }
                    if (half == 0 && c_ds > 0) {           // the previous dQ update has read dS
                        ok = wait(B_DSFREE, c_ds - 1u);
                        if (!ok) break;
                        tc_fence_after_sync();
                    }
                    tmem_st_x16(tm_ds + half * 16, ds + half * 16);
                    tmem_wait_st();
                    tc_fence_before_sync();
                    // first instalment: its arrival must not sink below the second half's arithmetic
                    if (half == 0) lse2_h = mbar_arrive_warp_before(bar(B_PFULL), lse2_h);
                    else mbar_arrive_warp(bar(B_PFULL + 1));
                }
                if (!ok) break;
                ++c_ds;
            }
            if (!ok) break;
            // ---- epilogue: dQ * scale -> bf16; this warpgroup writes half of the columns ---------
            ok = wait(B_DSFREE, c_ds - 1u);
            if (!ok) break;
            tc_fence_after_sync();
#pragma unroll
            for (int c0 = 0; c0 < kDqk / 2; c0 += 32) {
                uint32_t v[32];
                tmem_ld_x32(tm + kTmDQ + lane_base + g * (kDqk / 2) + c0, v);
                tmem_wait_ld();
                if (c0 + 32 == kDqk / 2) {
                    tc_fence_before_sync();
                    mbar_arrive_warp(bar(B_ACCFREE));
                }
                if (row_valid) {
                    if (p.accumulate) add_row_f32(dst_acc + c0, v, 32, p.scale);
                    else store_row_bf16(dst + c0, v, 32, p.scale);
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    if (abort_flag) {
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 50000ull) { }
        if (tid == 0) {
            p.status->detail = blockIdx.x;
            p.status->status = HYDRA_ERR_DEVICE_TIMEOUT;
        }
        __syncthreads();
    }
    if (warp == kWarpMma) tmem_dealloc(tm, kTmCols);
}

// =============================================================================================
// dK / dV
// =============================================================================================
__global__ void __launch_bounds__(kThreads, 1)
HYDRA_K(hydra_bwd_dkv_kernel)(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do,
                     const BwdParams p)
{
    using namespace dkv;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem = (smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t bars[B_COUNT];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ int32_t s_sched[kSched];
    __shared__ GroupItem s_item[kSched];              // the work ring carries the item and its first pair, so that
    __shared__ PairDev s_first[kSched];               // no role starts an item with a walk through global memory
    // -LSE * log2(e) and -D of the q rows of a sub-tile (negated by the producer: they are addends of packed
    // two-element operations, which have no operand negation; 16-byte aligned: read four columns at a time)
    __shared__ __align__(16) float s_lse2[kStages][SUB];
    __shared__ __align__(16) float s_dsum[kStages][SUB];
    __shared__ uint32_t s_bursts;                      // S / dP bursts issued so far (all ones: no more)

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t bar0 = smem_u32(&bars[0]);
    auto bar = [&](int i) -> uint32_t { return bar0 + 8u * static_cast<uint32_t>(i); };
    if (tid == 0) {
        abort_flag = 0;
        s_bursts = 0u;
        for (int i = 0; i < B_COUNT; ++i) {
            uint32_t count = 1u;
            if (i == B_SFREE || i == B_PFULL || i == B_ACCFREE) count = 8u;   // elementwise warps
            if (i >= B_ITEMEMPTY && i < B_ITEMEMPTY + kSched) count = 10u;   // + the two issuer warps
            
            mbar_init(bar(i), count);
        }
        fence_mbar_init();
        tma_prefetch_desc(&map_q); tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v); tma_prefetch_desc(&map_do);
    }
    if (warp == kWarpMma) { tmem_alloc(smem_u32(&tmem_base_slot), kTmCols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_base_slot;
    const uint64_t limit = p.wait_limit_ns;
    volatile int* abort_p = &abort_flag;
    auto wait = [&](int b, uint32_t parity) -> bool { return mbar_wait(bar(b), parity & 1u, abort_p, limit); };
    // Work queue: the producer pops the next item index from a counter in global memory (so a CTA that
    // finishes early simply takes more items: no cost model has to predict the run time of an item)
    // and hands it to the other warps of the CTA through a small ring in shared memory.
    volatile int32_t* sched = s_sched;
    // The pop is split in two: the request to the counter goes out when an item starts, its answer is
    // looked at after the first loads of that item have been issued; the producer then fetches the
    // next item's descriptors (three dependent loads from global memory) and puts them in the ring.
    constexpr int kPopFailed = 0x7fffffff;
    auto pop_begin = [&](uint32_t k) -> int {               // producer, one thread
        const int slot = k % kSched;
        if (!mbar_wait(bar(B_ITEMEMPTY + slot), ((k / kSched) ^ 1u) & 1u, abort_p, limit)) return kPopFailed;
        return atomicAdd(&p.status->next_item[QUEUE_DKV], 1);
    };
    auto pop_end = [&](uint32_t k, int raw, GroupItem& item_out, PairDev& first_out) -> int {
        if (raw == kPopFailed) return -1;
        const int slot = k % kSched;
        const int idx = raw >= p.n_items ? -1 : raw;
        if (idx >= 0) {
            item_out = p.items[idx];
            first_out = p.pairs[p.lists[item_out.list_off]];
            s_item[slot] = item_out;
            s_first[slot] = first_out;
        }
        sched[slot] = idx;
        mbar_arrive(bar(B_ITEMFULL + slot));
        return idx;
    };
    auto next_item = [&](uint32_t k, GroupItem& item_out, PairDev& first_out) -> int {   // every other warp, all lanes
        const int slot = k % kSched;
        if (!mbar_wait(bar(B_ITEMFULL + slot), (k / kSched) & 1u, abort_p, limit)) return -1;
        const int idx = sched[slot];
        if (idx >= 0) {
            item_out = s_item[slot];
            first_out = s_first[slot];
        }
        mbar_arrive_warp(bar(B_ITEMEMPTY + slot));
        return idx;
    };
    volatile uint32_t* bursts_p = &s_bursts;

    if (warp == kWarpProd) {
        // ------------------------------------------------------------------ TMA producer + LSE / D
        uint32_t items = 0, gq = 0;
        bool ok = true;
        int it_ahead = -1;
        ClockProbe probe;
        probe.start();
        GroupItem item_next;                          // lane 0: descriptors of the item popped ahead
        PairDev first_next;
        // test hook: idle, then hand out and load nothing; every other role's wait then runs out
        if (p.debug_stall_ns) {
            if (lane == 0) debug_stall(p.debug_stall_ns);
            __syncwarp();
            ok = false;
        }
        for (uint32_t kq = 0; ok; ++kq) {
            int it = 0, raw_next = 0;
            if (lane == 0) {                          // one pop per CTA, one item ahead, shared with the other lanes
                if (kq == 0) it_ahead = pop_end(0, pop_begin(0), item_next, first_next);
                it = it_ahead;
                if (it >= 0) raw_next = pop_begin(kq + 1);
            }
            bool popped = false;
            it = __shfl_sync(0xffffffffu, it, 0);
            if (it < 0) break;
            __syncwarp();
            // lane 0 wrote this item's descriptors into the ring when it popped it (before the barrier above)
            const GroupItem item = s_item[kq % kSched];
            const PairDev first = s_first[kq % kSched];
            const int32_t* list = p.lists + item.list_off;
            SubIter si;
            si.init(p.pairs, list, item.list_len, item.r0, p.causal, p.ds != nullptr, first);
            if (!si.valid()) {
                if (lane == 0) it_ahead = pop_end(kq + 1, raw_next, item_next, first_next);
                continue;
            }
            ok = wait(B_KVEMPTY, items ^ 1u);
            if (!ok) break;
            ++items;
            if (lane == 0) {
                mbar_arrive_expect_tx(bar(B_KVFULL), (kQkBoxes + 2) * kBox128);
                for (int c = 0; c < kQkBoxes; ++c)
                    tma_load_3d(smem + kK + c * kBox128, &map_k, bar(B_KVFULL), c * 64, item.head / p.kv_group,
                                first.k_tok0 + item.r0);
                for (int c = 0; c < 2; ++c)
                    tma_load_3d(smem + kV + c * kBox128, &map_v, bar(B_KVFULL), c * 64, item.head / p.kv_group,
                                first.k_tok0 + item.r0);
            }
            for (; si.valid() && ok; si.next(), ++gq) {
                const int st = gq % kStages;
                ok = wait(B_QEMPTY + st, (gq / kStages) ^ 1u);
                if (!ok) break;
                const int tok = si.cur.q_tok0 + si.u * SUB;
                if (lane == 0) {
                    mbar_arrive_expect_tx(bar(B_QFULL + st), (kQkBoxes + 2) * kBox64);
                    for (int c = 0; c < kQkBoxes; ++c)
                        tma_load_3d(smem + kQ + st * kQkBoxes * kBox64 + c * kBox64, &map_q, bar(B_QFULL + st), c * 64,
                                    item.head, tok);
                    for (int c = 0; c < 2; ++c)
                        tma_load_3d(smem + kDO + st * 2 * kBox64 + c * kBox64, &map_do, bar(B_QFULL + st), c * 64,
                                    item.head, tok);
                }
                // LSE (as log2) and D of the 64 q rows, two rows per lane
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int c = lane + 32 * e;
                    const int i = si.u * SUB + c;
                    const bool v = i < si.cur.q_len;
                    const int64_t idx = static_cast<int64_t>(item.head) * p.T + si.cur.q_tok0 + i;
                    const float l = v ? __ldg(p.lse + idx) : neg_inf();
                    s_lse2[st][c] = (l == neg_inf()) ? neg_inf() : -(l * kLog2e);
                    s_dsum[st][c] = v ? -__ldg(p.dsum + idx) : 0.f;
                }
                mbar_arrive_warp(bar(B_STAT + st));
                if (!popped) {
                    if (lane == 0) it_ahead = pop_end(kq + 1, raw_next, item_next, first_next);
                    popped = true;
                }
            }
            if (!popped && lane == 0) it_ahead = pop_end(kq + 1, raw_next, item_next, first_next);
        }
        if (blockIdx.x == 0 && lane == 0) probe.stop(p.status, QUEUE_DKV);
    } else if (warp == kWarpMma || warp == kWarpMma2) {
        // ------------------------------------------------------------------ UMMA issuers
        // warp 9 issues S^T = K Q^T and dP^T = V dO^T of sub-tile u+1 as soon as those of sub-tile u
        // have been copied out; warp 10 issues dV += P^T dO and dK += dS^T Q of sub-tile u as soon
        // as P and dS are in tensor memory. Neither waits behind the other's operands.
        // The whole warp walks the work list; one elected lane issues the UMMAs and commits.
        {
            constexpr uint32_t idesc_st = umma_idesc_bf16(TILE, SUB, false, false);
            constexpr uint32_t idesc_dv = umma_idesc_bf16(TILE, D_V, false, true);
            constexpr uint32_t idesc_dk = umma_idesc_bf16(TILE, kDqk, false, true);
            constexpr uint32_t hi_kmaj = umma_desc_hi(16, 1024);
            constexpr uint32_t hi_mn = umma_desc_hi(kBox64, 1024);         // Q / dO sub-tiles as MN-major B
            const uint32_t k_lo = umma_desc_lo(smem + kK, 16), v_lo = umma_desc_lo(smem + kV, 16);
            const uint32_t q_lo0 = umma_desc_lo(smem + kQ, 16), do_lo0 = umma_desc_lo(smem + kDO, 16);
            const uint32_t qmn_lo0 = umma_desc_lo(smem + kQ, kBox64), domn_lo0 = umma_desc_lo(smem + kDO, kBox64);
            const bool issue_scores = warp == kWarpMma;
            uint32_t items = 0, n_step = 0;
            bool ok = true;
            for (uint32_t kq = 0; ok; ++kq) {
                GroupItem item;
                PairDev first;
                const int it = next_item(kq, item, first);
                if (it < 0) break;
                const int32_t* list = p.lists + item.list_off;
                SubIter si;
                si.init(p.pairs, list, item.list_len, item.r0, p.causal, p.ds != nullptr, first);
                if (!si.valid()) continue;
                if (issue_scores) {
                    ok = wait(B_KVFULL, items);
                    for (; si.valid() && ok;) {
                        // the poll that is almost always satisfied (Q / dO landed stages ago) and the
                        // address arithmetic come first; the wait on the critical path (S / dP of the
                        // previous sub-tile copied out) comes last, with only the UMMAs behind it
                        const int st = n_step % kStages;
                        ok = wait(B_QFULL + st, n_step / kStages);
                        if (!ok) break;
                        const uint32_t q_lo = q_lo0 + st * (kQkBoxes * kBox64 >> 4), do_lo = do_lo0 + st * (2 * kBox64 >> 4);
                        const uint32_t prev = n_step;
                        ++n_step;
                        si.next();
                        if (prev > 0) ok = wait(B_SFREE, prev - 1u);
                        if (!ok) break;
                        tc_fence_after_sync();
                        if (elect_one()) {
#pragma unroll
                            for (int kk = 0; kk < kDqk / 16; ++kk)
                                umma_ss_w(tm + kTmS, k_lo + (kk >> 2) * (kBox128 >> 4) + (kk & 3) * 2, hi_kmaj,
                                          q_lo + (kk >> 2) * (kBox64 >> 4) + (kk & 3) * 2, hi_kmaj, idesc_st, kk > 0);
#pragma unroll
                            for (int kk = 0; kk < D_V / 16; ++kk)
                                umma_ss_w(tm + kTmDP, v_lo + (kk >> 2) * (kBox128 >> 4) + (kk & 3) * 2, hi_kmaj,
                                          do_lo + (kk >> 2) * (kBox64 >> 4) + (kk & 3) * 2, hi_kmaj, idesc_st, kk > 0);
                            umma_commit(bar(B_SFULL));
                            *bursts_p = n_step;
                            if (!si.valid()) umma_commit(bar(B_KVEMPTY));    // K and V are no longer read
                        }
                    }
                } else {
                    bool first_step = true;
                    for (; si.valid() && ok; si.next()) {
                        ok = wait(B_PFULL, n_step);
                        if (ok && first_step && items > 0) ok = wait(B_ACCFREE, items - 1u);
                        // Order hint, not a data dependency: let the score products of the NEXT sub-tile of
                        // this item enter the tensor pipe first. They are what the elementwise warps wait
                        // for next; these updates then fill the gap in which S / dP are copied out,
                        // instead of interleaving with the score products and delaying them.
                        SubIter peek = si;
                        peek.next();
                        if (ok && peek.valid()) ok = counter_wait(bursts_p, n_step + 2u, abort_p, limit);
                        if (!ok) break;
                        tc_fence_after_sync();
                        const int st = n_step % kStages;
                        const uint32_t do_lo = domn_lo0 + st * (2 * kBox64 >> 4), q_lo = qmn_lo0 + st * (kQkBoxes * kBox64 >> 4);
                        const uint32_t acc = first_step ? 0u : 1u;
                        if (elect_one()) {
#pragma unroll
                            for (int kk = 0; kk < SUB / 16; ++kk)
                                umma_ts_w(tm + kTmDV, tm + kTmP + kk * 8, do_lo + kk * (2048 >> 4), hi_mn, idesc_dv,
                                          kk > 0 ? 1u : acc);
#pragma unroll
                            for (int kk = 0; kk < SUB / 16; ++kk)
                                umma_ts_w(tm + kTmDK, tm + kTmDS + kk * 8, q_lo + kk * (2048 >> 4), hi_mn, idesc_dk,
                                          kk > 0 ? 1u : acc);
                            umma_commit(bar(B_PDSFREE));
                            umma_commit(bar(B_QEMPTY + st));
                        }
                        ++n_step;
                        first_step = false;
                    }
                }
                ++items;
            }
            if (issue_scores && elect_one()) *bursts_p = 0xffffffffu;         // nothing more to wait for
        }
    } else {
        // ------------------------------------------------------------------ elementwise warpgroups
        const int g = warp >> 2;                       // column half: q rows [32 g, 32 g + 32) of the sub-tile
        const int r = tid & 127;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tm_s = tm + kTmS + lane_base + g * 32;
        const uint32_t tm_dp = tm + kTmDP + lane_base + g * 32;
        const uint32_t tm_p = tm + kTmP + lane_base + g * 16;
        const uint32_t tm_ds = tm + kTmDS + lane_base + g * 16;
        uint32_t c_s = 0, c_pds = 0, gq = 0;
        int ds_li = -1;                                // pair whose first hand-off block is in ds_blk0
        int64_t ds_blk0 = 0;
        bool ok = true;
        for (uint32_t kq = 0; ok; ++kq) {
            GroupItem item;
            PairDev first;
            const int it = next_item(kq, item, first);
            if (it < 0) break;
            const int32_t* list = p.lists + item.list_off;
            ds_li = -1;
            const int krow = item.r0 + r;              // kv row inside the chunk
            const bool row_valid = krow < first.k_len;
            const int64_t tok = static_cast<int64_t>(first.k_tok0) + krow;
            // with shared KV heads (accumulating form only) the query heads of a group add into one dk / dv row
            const int64_t kv_heads = p.h / p.kv_group;
            const int64_t kv_row = tok * kv_heads + item.head / p.kv_group;
            const int64_t dk_off = kv_row * kDqk + g * (kDqk / 2);
            const int64_t dv_off = kv_row * D_V + g * 64;
            __nv_bfloat16* dkp = static_cast<__nv_bfloat16*>(p.dk) + dk_off;
            __nv_bfloat16* dvp = static_cast<__nv_bfloat16*>(p.dv) + dv_off;
            float* dkp_acc = static_cast<float*>(p.dk) + dk_off;         // accumulate mode: dk, dv are fp32
            float* dvp_acc = static_cast<float*>(p.dv) + dv_off;
            SubIter si;
            si.init(p.pairs, list, item.list_len, item.r0, p.causal, p.ds != nullptr, first);
            if (!si.valid()) {                         // no q row sees this tile: dK = dV = 0 (nothing to add)
                if (row_valid && !p.accumulate) {
                    uint4* a4 = reinterpret_cast<uint4*>(dkp);
                    uint4* b4 = reinterpret_cast<uint4*>(dvp);
#pragma unroll
                    for (int e = 0; e < kDqk / 16; ++e) a4[e] = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                    for (int e = 0; e < 8; ++e) b4[e] = make_uint4(0u, 0u, 0u, 0u);
                }
                continue;
            }
            for (; si.valid() && ok; si.next(), ++gq) {
                const int st = gq % kStages;
                ok = wait(B_SFULL, c_s);
                ++c_s;
                if (!ok) break;
                tc_fence_after_sync();
                uint32_t s[32], dp[32];
                tmem_ld_x32(tm_s, s);
                tmem_ld_x32(tm_dp, dp);
                tmem_wait_ld();
                tc_fence_before_sync();
                mbar_arrive_warp(bar(B_SFREE));
                ok = wait(B_STAT + st, gq / kStages);
                if (!ok) break;
                // q row i = u*64 + 32 g + c is visible from kv row krow iff i < q_len and krow <= i + off
                const int base = si.u * SUB + g * 32;
                int c_lo = 0;
                if (p.causal) c_lo = max(0, krow - si.cur.off - base);
                int c_hi = min(32, si.cur.q_len - base);
                if (!row_valid) c_hi = 0;
                const float4* nlse4 = reinterpret_cast<const float4*>(&s_lse2[st][g * 32]);
                const float4* ndsum4 = reinterpret_cast<const float4*>(&s_dsum[st][g * 32]);
                uint32_t pk[16], ds[16];
                // Interior sub-tiles (every q row visible from every kv row of the warp) skip the masking; elsewhere
                // the masked scores become -inf, whose probability exp2(-inf) is 0 by itself: one arithmetic path.
                if (__any_sync(0xffffffffu, c_lo > 0 || c_hi < 32)) {
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (c < c_lo || c >= c_hi) s[c] = __float_as_uint(neg_inf());
                }
#pragma unroll
                for (int c = 0; c < 32; c += 4) {
                    const float4 nl = nlse4[c >> 2], nd = ndsum4[c >> 2];
                    const float nlv[4] = {nl.x, nl.y, nl.z, nl.w}, ndv[4] = {nd.x, nd.y, nd.z, nd.w};
#pragma unroll
                    for (int e = 0; e < 4; e += 2) {
                        float x0, x1, d0, d1;
                        ffma2(x0, x1, __uint_as_float(s[c + e]), __uint_as_float(s[c + e + 1]), p.scale_log2,
                              p.scale_log2, nlv[e], nlv[e + 1]);
                        const float p0 = ex2_approx(x0), p1 = ex2_approx(x1);
                        fadd2(d0, d1, __uint_as_float(dp[c + e]), __uint_as_float(dp[c + e + 1]), ndv[e], ndv[e + 1]);
                        fmul2(d0, d1, d0, d1, p0, p1);
                        pk[(c + e) >> 1] = pack_bf16x2(p0, p1);
                        ds[(c + e) >> 1] = pack_bf16x2(d0, d1);
                    }
                }
                if (c_pds > 0) {                       // the previous dV / dK updates have read P and dS
                    ok = wait(B_PDSFREE, c_pds - 1u);
                    if (!ok) break;
                    tc_fence_after_sync();
                }
                tmem_st_x16(tm_p, pk);
                tmem_st_x16(tm_ds, ds);
                tmem_wait_st();
                tc_fence_before_sync();
                mbar_arrive_warp(bar(B_PFULL));
                ++c_pds;
                if (p.ds) {
                    // Hand dS^T to the query-side kernel (after P and dS have gone to the tensor core: off the
                    // chain S -> P, dS -> dV, dK).
                    if (si.li != ds_li) {
                        ds_li = si.li;
                        const DsGeom geo = ds_geom(si.cur.q_len, si.cur.off, p.causal);
                        const int jk = item.r0 / TILE;
                        ds_blk0 = static_cast<int64_t>(item.head) * p.ds_head_blocks + si.cur.ds_base +
                                  ds_rowstart(geo, jk) - ds_first(geo, jk);
                    }
                    // The block in memory is 8 chunks (8 q rows each) of 128 kv rows x 16 bytes: lane = kv row,
                    // so every store instruction of the warp writes 512 contiguous bytes.
                    uint8_t* blk = static_cast<uint8_t*>(p.ds) + (ds_blk0 + si.u) * DS_BLOCK_BYTES + g * 4 * 2048 +
                                   ((warp & 3) * 32 + lane) * 16;
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        st_global_stream_v4(blk + e * 2048,
                                            make_uint4(ds[4 * e], ds[4 * e + 1], ds[4 * e + 2], ds[4 * e + 3]));
                }
            }
            if (!ok) break;
            // ---- epilogue: dK * scale, dV -> bf16; each warpgroup writes half of the columns -------
            ok = wait(B_PDSFREE, c_pds - 1u);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t rows_valid = __ballot_sync(0xffffffffu, row_valid);
            const uint32_t out_slice = smem + kDsStage + warp * 2048;
            // chunks of 32 columns (dK: kDkChunks, then dV: 2); the load of the next chunk is in flight while
            // the current one is packed, transposed and stored
            constexpr int kDkChunks = kDqk / 64, kChunks = kDkChunks + 2;
            auto chunk_addr = [&](int c) -> uint32_t {
                return c < kDkChunks ? tm + kTmDK + lane_base + g * (kDqk / 2) + c * 32
                                     : tm + kTmDV + lane_base + g * 64 + (c - kDkChunks) * 32;
            };
            uint32_t va[32], vb[32];
            tmem_ld_x32(chunk_addr(0), va);
#pragma unroll
            for (int c = 0; c < kChunks; ++c) {
                uint32_t* cur = (c & 1) ? vb : va;
                uint32_t* nxt = (c & 1) ? va : vb;
                tmem_wait_ld();
                if (c + 1 < kChunks) tmem_ld_x32(chunk_addr(c + 1), nxt);
                if (c == kChunks - 1) {                          // every column has left tensor memory
                    tc_fence_before_sync();
                    mbar_arrive_warp(bar(B_ACCFREE));
                }
                const bool is_dk = c < kDkChunks;
                const int c0 = is_dk ? c * 32 : (c - kDkChunks) * 32;
                if (p.accumulate) {
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        if (is_dk)
                            add_rows_f32_coalesced(out_slice, lane, dkp_acc + c0 + half * 16, kv_heads * kDqk,
                                                   cur + half * 16, p.scale, rows_valid);
                        else
                            add_rows_f32_coalesced(out_slice, lane, dvp_acc + c0 + half * 16, kv_heads * D_V,
                                                   cur + half * 16, 1.f, rows_valid);
                    }
                } else if (is_dk) {
                    store_rows_bf16_coalesced(out_slice, lane, dkp + c0, kv_heads * kDqk, cur, p.scale, rows_valid);
                } else {
                    store_rows_bf16_coalesced(out_slice, lane, dvp + c0, kv_heads * D_V, cur, 1.f, rows_valid);
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    if (abort_flag) {
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 50000ull) { }
        if (tid == 0) {
            p.status->detail = blockIdx.x;
            p.status->status = HYDRA_ERR_DEVICE_TIMEOUT;
        }
        __syncthreads();
    }
    if (warp == kWarpMma) tmem_dealloc(tm, kTmCols);
}

// =============================================================================================
// dQ from the dS hand-off buffer
// =============================================================================================
// When the key-side kernel has left dS^T in memory, dQ = scale * dS K needs no recomputation of S
// and dP: per (q tile, kv tile) one product of 128 x 192 x 128, both operands as they arrive (the dS^T
// blocks, stored by the key-side kernel in the unswizzled MN-major operand layout, as the A operand; the K
// tile from its swizzled TMA boxes as an MN-major B operand). The kernel is
// bound by the stream of dS (2 bytes per 384 FLOP), so it is a plain load -> UMMA -> store pipeline:
//   warps 0-3  epilogue (thread r = q row r): dQ * scale -> bf16 (or fp32 reductions), rows transposed
//              through 2 KB of shared memory per warp so that whole 64-byte segments are stored
//   warp  4    pops work items; producer of dS^T: per kv tile the two adjacent blocks of the q tile as one
//              untiled 32 KB bulk copy, ring of three (dS comes from memory)
//   warp  5    UMMA issuer; two accumulators in tensor memory, so the epilogue of one work item
//              overlaps the products of the next
//   warp  6    TMA producer of the K tiles (48 KB, ring of two: they come from the L2 cache)
// Per SM the kernel is bound by what TMA can bring in (80 KB per 768 cycles of UMMA).
namespace dqs {
constexpr int kThreadsS = 224;
constexpr int kDsStages = 3, kKStages = 2;
constexpr uint32_t kDsBytes = 2 * DS_BLOCK_BYTES;            // blocks (jk, 2i) and (jk, 2i + 1)
constexpr uint32_t kK = kDsStages * kDsBytes;                // 96 KB of dS^T, then the K tiles
constexpr uint32_t kOut = kK + kKStages * kQkBoxes * kBox128;       // 4 epilogue warps x 2 KB: dQ rows on their way out
constexpr uint32_t kTotal = kOut + 4 * 2048;                 // 204,800 B at d_qk = 192
constexpr uint32_t kTmAcc = 256, kTmCols = 512;              // accumulators at columns 0 and 256
enum : int { B_DSFULL = 0, B_DSEMPTY = 4, B_KFULL = 8, B_KEMPTY = 10, B_ACCFULL = 12, B_ACCFREE = 14,
             B_ITEMFULL = 16, B_ITEMEMPTY = 16 + kSched, B_COUNT = 16 + 2 * kSched };
}  // namespace dqs

size_t HYDRA_K(bwd_dq_ds_smem_bytes)() { return dqs::kTotal + 1024; }

__global__ void __launch_bounds__(dqs::kThreadsS, 1)
HYDRA_K(hydra_bwd_dq_from_ds_kernel)(const __grid_constant__ CUtensorMap map_k,
                            const BwdParams p)
{
    using namespace dqs;
    using dq::TileIter;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem = (smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t bars[B_COUNT];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ int32_t s_sched[kSched];
    __shared__ GroupItem s_item[kSched];              // the work ring carries the item and its first pair, so that
    __shared__ PairDev s_first[kSched];               // no role starts an item with a walk through global memory

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t bar0 = smem_u32(&bars[0]);
    auto bar = [&](int i) -> uint32_t { return bar0 + 8u * static_cast<uint32_t>(i); };
    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < B_COUNT; ++i) {
            uint32_t count = 1u;
            if (i == B_ACCFREE || i == B_ACCFREE + 1) count = 4u;             // epilogue warps
            if (i >= B_ITEMEMPTY && i < B_ITEMEMPTY + kSched) count = 6u;    // + issuer and K producer warps
            mbar_init(bar(i), count);
        }
        fence_mbar_init();
        tma_prefetch_desc(&map_k);
    }
    if (warp == 5) { tmem_alloc(smem_u32(&tmem_base_slot), kTmCols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_base_slot;
    const uint64_t limit = p.wait_limit_ns;
    volatile int* abort_p = &abort_flag;
    auto wait = [&](int b, uint32_t parity) -> bool { return mbar_wait(bar(b), parity & 1u, abort_p, limit); };
    volatile int32_t* sched = s_sched;
    // The pop is split in two: the request to the counter goes out when an item starts, its answer is
    // looked at after the first loads of that item have been issued; the producer then fetches the
    // next item's descriptors (three dependent loads from global memory) and puts them in the ring.
    constexpr int kPopFailed = 0x7fffffff;
    auto pop_begin = [&](uint32_t k) -> int {               // producer, one thread
        const int slot = k % kSched;
        if (!mbar_wait(bar(B_ITEMEMPTY + slot), ((k / kSched) ^ 1u) & 1u, abort_p, limit)) return kPopFailed;
        return atomicAdd(&p.status->next_item[QUEUE_DQ], 1);
    };
    auto pop_end = [&](uint32_t k, int raw, GroupItem& item_out, PairDev& first_out) -> int {
        if (raw == kPopFailed) return -1;
        const int slot = k % kSched;
        const int idx = raw >= p.n_items ? -1 : raw;
        if (idx >= 0) {
            item_out = p.items[idx];
            first_out = p.pairs[p.lists[item_out.list_off]];
            s_item[slot] = item_out;
            s_first[slot] = first_out;
        }
        sched[slot] = idx;
        mbar_arrive(bar(B_ITEMFULL + slot));
        return idx;
    };
    auto next_item = [&](uint32_t k, GroupItem& item_out, PairDev& first_out) -> int {   // every other warp, all lanes
        const int slot = k % kSched;
        if (!mbar_wait(bar(B_ITEMFULL + slot), (k / kSched) & 1u, abort_p, limit)) return -1;
        const int idx = sched[slot];
        if (idx >= 0) {
            item_out = s_item[slot];
            first_out = s_first[slot];
        }
        mbar_arrive_warp(bar(B_ITEMEMPTY + slot));
        return idx;
    };

    if (warp == 4) {
        // ------------------------------------------------------------------ work queue + dS producer
        if (lane == 0) {
            uint32_t g = 0;
            bool ok = true;
            const uint64_t ds_policy = l2_policy_evict_first();   // dS is read once: leave L2 to the K tiles
            ClockProbe probe;
            probe.start();
            GroupItem item_next;
            PairDev first_next;
            // test hook: idle, then hand out and load nothing; every other role's wait then runs out
            if (p.debug_stall_ns) { debug_stall(p.debug_stall_ns); ok = false; }
            int it_ahead = ok ? pop_end(0, pop_begin(0), item_next, first_next) : -1;
            for (uint32_t kq = 0; ok; ++kq) {
                const int it = it_ahead;
                if (it < 0) break;
                const GroupItem item = item_next;
                const PairDev first = first_next;
                const int raw_next = pop_begin(kq + 1);
                bool popped = false;
                const int32_t* list = p.lists + item.list_off;
                TileIter ti;
                ti.init(p.pairs, list, item.list_len, min(item.r0 + TILE, first.q_len) - 1, p.causal, first);
                const int u0 = item.r0 / SUB;                  // first sub-tile of this q tile
                for (; ti.valid() && ok; ti.next(), ++g) {
                    const int st = g % kDsStages;
                    ok = wait(B_DSEMPTY + st, (g / kDsStages) ^ 1u);
                    if (!ok) break;
                    const DsGeom geo = ds_geom(ti.cur.q_len, ti.cur.off, p.causal);
                    const int64_t blk = static_cast<int64_t>(item.head) * p.ds_head_blocks + ti.cur.ds_base +
                                        ds_rowstart(geo, ti.t) + (u0 - ds_first(geo, ti.t));
                    mbar_arrive_expect_tx(bar(B_DSFULL + st), kDsBytes);
                    bulk_load_hint(smem + st * kDsBytes, static_cast<const uint8_t*>(p.ds) + blk * DS_BLOCK_BYTES,
                                   kDsBytes, bar(B_DSFULL + st), ds_policy);
                    if (!popped) { it_ahead = pop_end(kq + 1, raw_next, item_next, first_next); popped = true; }
                }
                if (!popped) it_ahead = pop_end(kq + 1, raw_next, item_next, first_next);
            }
            if (blockIdx.x == 0) probe.stop(p.status, QUEUE_DQ);
        }
    } else if (warp == 6) {
        // ------------------------------------------------------------------ K producer
        uint32_t g = 0;
        bool ok = true;
        for (uint32_t kq = 0; ok; ++kq) {
            GroupItem item;
            PairDev first;
            const int it = next_item(kq, item, first);
            if (it < 0) break;
            const int32_t* list = p.lists + item.list_off;
            TileIter ti;
            ti.init(p.pairs, list, item.list_len, min(item.r0 + TILE, first.q_len) - 1, p.causal, first);
            for (; ti.valid() && ok; ti.next(), ++g) {
                const int st = g % kKStages;
                ok = wait(B_KEMPTY + st, (g / kKStages) ^ 1u);
                if (!ok) break;
                if (lane == 0) {
                    mbar_arrive_expect_tx(bar(B_KFULL + st), kQkBoxes * kBox128);
                    for (int c = 0; c < kQkBoxes; ++c)
                        tma_load_3d(smem + kK + (st * kQkBoxes + c) * kBox128, &map_k, bar(B_KFULL + st), c * 64,
                                    item.head / p.kv_group, ti.cur.k_tok0 + ti.t * TILE);
                }
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------------ UMMA issuer
        constexpr uint32_t idesc = umma_idesc_bf16(TILE, kDqk, true, true);
        // dS^T without swizzle: 8 kv rows are 128 bytes, chunks of 8 q rows are 2 KB apart (two blocks in a row)
        constexpr uint32_t hi_ds = umma_desc_plain_hi(128, 2048);
        constexpr uint32_t hi_k = umma_desc_hi(kBox128, 1024);           // K: N chunks of 64 columns 16 KB apart
        uint32_t g = 0, n_acc = 0;
        bool ok = true;
        for (uint32_t kq = 0; ok; ++kq) {
            GroupItem item;
            PairDev first;
            const int it = next_item(kq, item, first);
            if (it < 0) break;
            const int32_t* list = p.lists + item.list_off;
            TileIter ti;
            ti.init(p.pairs, list, item.list_len, min(item.r0 + TILE, first.q_len) - 1, p.causal, first);
            if (!ti.valid()) continue;
            const uint32_t buf = n_acc & 1u;
            ok = wait(B_ACCFREE + buf, (n_acc >> 1) ^ 1u);
            if (!ok) break;
            bool first_tile = true;
            for (; ti.valid() && ok; ti.next(), ++g) {
                const int ds_st = g % kDsStages, k_st = g % kKStages;
                ok = wait(B_KFULL + k_st, g / kKStages);
                if (ok) ok = wait(B_DSFULL + ds_st, g / kDsStages);
                if (!ok) break;
                tc_fence_after_sync();
                if (elect_one()) {
                    const uint32_t a_lo = umma_desc_plain_lo(smem + ds_st * kDsBytes, 128);
                    const uint32_t b_lo = umma_desc_lo(smem + kK + k_st * kQkBoxes * kBox128, kBox128);
#pragma unroll
                    for (int kk = 0; kk < TILE / 16; ++kk)
                        umma_ss_w(tm + buf * kTmAcc, a_lo + kk * (256 >> 4), hi_ds, b_lo + kk * (2048 >> 4), hi_k, idesc,
                                  (kk > 0 || !first_tile) ? 1u : 0u);
                    umma_commit(bar(B_DSEMPTY + ds_st));
                    umma_commit(bar(B_KEMPTY + k_st));
                }
                first_tile = false;
            }
            if (ok && elect_one()) umma_commit(bar(B_ACCFULL + buf));
            __syncwarp();
            ++n_acc;
        }
    } else if (warp < 4) {
        // ------------------------------------------------------------------ epilogue warps
        const int r = tid;                             // q row inside the tile = TMEM lane
        const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
        uint32_t n_acc = 0;
        bool ok = true;
        for (uint32_t kq = 0; ok; ++kq) {
            GroupItem item;
            PairDev first;
            const int it = next_item(kq, item, first);
            if (it < 0) break;
            const int32_t* list = p.lists + item.list_off;
            const int row = item.r0 + r;
            const bool row_valid = row < first.q_len;
            const int64_t dst_off = (static_cast<int64_t>(first.q_tok0 + row) * p.h + item.head) * kDqk;
            __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(p.dq) + dst_off;
            float* dst_acc = static_cast<float*>(p.dq) + dst_off;
            TileIter ti;
            ti.init(p.pairs, list, item.list_len, min(item.r0 + TILE, first.q_len) - 1, p.causal, first);
            if (!ti.valid()) {                         // no visible key at all: dQ = 0 (nothing to add)
                if (row_valid && !p.accumulate) {
                    uint4* d4 = reinterpret_cast<uint4*>(dst);
#pragma unroll
                    for (int e = 0; e < kDqk / 8; ++e) d4[e] = make_uint4(0u, 0u, 0u, 0u);
                }
                continue;
            }
            const uint32_t buf = n_acc & 1u;
            ok = wait(B_ACCFULL + buf, n_acc >> 1);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t rows_valid = __ballot_sync(0xffffffffu, row_valid);
            const uint32_t out_slice = smem + kOut + warp * 2048;
#pragma unroll
            for (int c0 = 0; c0 < kDqk; c0 += 32) {
                uint32_t v[32];
                tmem_ld_x32(tm + buf * kTmAcc + lane_base + c0, v);
                tmem_wait_ld();
                if (c0 + 32 == kDqk) {
                    tc_fence_before_sync();
                    mbar_arrive_warp(bar(B_ACCFREE + buf));
                }
                if (p.accumulate) {
#pragma unroll
                    for (int half = 0; half < 2; ++half)
                        add_rows_f32_coalesced(out_slice, lane, dst_acc + c0 + half * 16, static_cast<int64_t>(p.h) * kDqk,
                                               v + half * 16, p.scale, rows_valid);
                } else {
                    store_rows_bf16_coalesced(out_slice, lane, dst + c0, static_cast<int64_t>(p.h) * kDqk, v, p.scale, rows_valid);
                }
            }
            ++n_acc;
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    if (abort_flag) {
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 50000ull) { }
        if (tid == 0) {
            p.status->detail = blockIdx.x;
            p.status->status = HYDRA_ERR_DEVICE_TIMEOUT;
        }
        __syncthreads();
    }
    if (warp == 5) tmem_dealloc(tm, kTmCols);
}


// cudaFuncSetAttribute applies to the device that is current when it is called, so the opt-in to more than
// 48 KB of dynamic shared memory is made once per device ordinal, not once per process.
template <class Kernel>
cudaError_t configure_once_per_device(Kernel kernel, size_t smem_bytes, bool (&done)[64])
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (done[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_bytes));
    if (e == cudaSuccess) done[dev] = true;
    return e;
}

cudaError_t HYDRA_K(launch_bwd_dq_from_ds)(const CUtensorMap& mk, const BwdParams& p, int grid,
                                  cudaStream_t stream)
{
    static bool configured[64] = {};
    if (cudaError_t e = configure_once_per_device(HYDRA_K(hydra_bwd_dq_from_ds_kernel), HYDRA_K(bwd_dq_ds_smem_bytes)(), configured)) return e;
    HYDRA_K(hydra_bwd_dq_from_ds_kernel)<<<grid, dqs::kThreadsS, HYDRA_K(bwd_dq_ds_smem_bytes)(), stream>>>(mk, p);
    return cudaGetLastError();
}

cudaError_t HYDRA_K(launch_bwd_dq)(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                          const CUtensorMap& mdo, const BwdParams& p, int grid, cudaStream_t stream)
{
    static bool configured[64] = {};
    if (cudaError_t e = configure_once_per_device(HYDRA_K(hydra_bwd_dq_kernel), HYDRA_K(bwd_dq_smem_bytes)(), configured)) return e;
    HYDRA_K(hydra_bwd_dq_kernel)<<<grid, kThreads, HYDRA_K(bwd_dq_smem_bytes)(), stream>>>(mq, mk, mv, mdo, p);
    return cudaGetLastError();
}

cudaError_t HYDRA_K(launch_bwd_dkv)(const CUtensorMap& mq_sub, const CUtensorMap& mk, const CUtensorMap& mv,
                           const CUtensorMap& mdo_sub, const BwdParams& p, int grid, cudaStream_t stream)
{
    static bool configured[64] = {};
    if (cudaError_t e = configure_once_per_device(HYDRA_K(hydra_bwd_dkv_kernel), HYDRA_K(bwd_dkv_smem_bytes)(), configured)) return e;
    HYDRA_K(hydra_bwd_dkv_kernel)<<<grid, kThreads, HYDRA_K(bwd_dkv_smem_bytes)(), stream>>>(mq_sub, mk, mv, mdo_sub, p);
    return cudaGetLastError();
}

}  // namespace hydra
