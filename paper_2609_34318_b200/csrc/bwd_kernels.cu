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
#include <cuda_bf16.h>

#include "hydra_internal.h"
#include "sm100_ptx.cuh"

namespace hydra {

namespace {

constexpr int kThreads = 128;
constexpr uint32_t kBox128 = 128 * 128;   // [128 rows x 64 bf16]
constexpr uint32_t kBox64 = 64 * 128;     // [ 64 rows x 64 bf16]

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }
__device__ __forceinline__ float pos_inf() { return __int_as_float(0x7f800000); }

__device__ __forceinline__ void store_row_bf16(__nv_bfloat16* dst, const uint32_t* v, int n, float mul)
{
    uint4* d4 = reinterpret_cast<uint4*>(dst);
#pragma unroll
    for (int e = 0; e < n; e += 8) {
        uint4 w;
        w.x = pack_bf16x2(__uint_as_float(v[e + 0]) * mul, __uint_as_float(v[e + 1]) * mul);
        w.y = pack_bf16x2(__uint_as_float(v[e + 2]) * mul, __uint_as_float(v[e + 3]) * mul);
        w.z = pack_bf16x2(__uint_as_float(v[e + 4]) * mul, __uint_as_float(v[e + 5]) * mul);
        w.w = pack_bf16x2(__uint_as_float(v[e + 6]) * mul, __uint_as_float(v[e + 7]) * mul);
        d4[e >> 3] = w;
    }
}

// ---------------------------------------------------------------------------------------------
// dQ kernel
// ---------------------------------------------------------------------------------------------
namespace dq {
constexpr uint32_t kQ = 0;                          // 3 boxes
constexpr uint32_t kDO = kQ + 3 * kBox128;          // 2 boxes
constexpr uint32_t kK = kDO + 2 * kBox128;          // 2 stages x 3 boxes
constexpr uint32_t kV = kK + 2 * 3 * kBox128;       // 1 stage x 2 boxes
constexpr uint32_t kTotal = kV + 2 * kBox128;       // 212,992 B
constexpr uint32_t kTmS = 0, kTmDP = 128, kTmDQ = 256, kTmDS = 448, kTmCols = 512;
}  // namespace dq

// ---------------------------------------------------------------------------------------------
// dK/dV kernel
// ---------------------------------------------------------------------------------------------
namespace dkv {
constexpr uint32_t kK = 0;                          // 3 boxes of 128 rows
constexpr uint32_t kV = kK + 3 * kBox128;           // 2 boxes of 128 rows
constexpr uint32_t kQ = kV + 2 * kBox128;           // 2 stages x 3 boxes of 64 rows
constexpr uint32_t kDO = kQ + 2 * 3 * kBox64;       // 2 stages x 2 boxes of 64 rows
constexpr uint32_t kTotal = kDO + 2 * 2 * kBox64;   // 163,840 B
constexpr uint32_t kTmDK = 0, kTmDV = 192, kTmS = 320, kTmDP = 384, kTmP = 448, kTmDS = 480,
                   kTmCols = 512;
}  // namespace dkv

}  // namespace

size_t bwd_dq_smem_bytes() { return dq::kTotal + 1024; }
size_t bwd_dkv_smem_bytes() { return dkv::kTotal + 1024; }

__global__ void __launch_bounds__(kThreads, 1)
hydra_bwd_dq_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do,
                    const BwdParams p)
{
    using namespace dq;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem = (smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t bars[8];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5;
    const uint32_t bar_q = smem_u32(&bars[0]);      // Q and dO of the item
    const uint32_t bar_k0 = smem_u32(&bars[1]);     // + 8 * stage
    const uint32_t bar_v = smem_u32(&bars[3]);
    const uint32_t bar_s = smem_u32(&bars[4]);      // S and dP complete
    const uint32_t bar_acc = smem_u32(&bars[5]);    // dQ += dS K complete

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(bar_q, 1); mbar_init(bar_k0, 1); mbar_init(bar_k0 + 8, 1);
        mbar_init(bar_v, 1); mbar_init(bar_s, 1); mbar_init(bar_acc, 1);
        fence_mbar_init();
        tma_prefetch_desc(&map_q); tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v); tma_prefetch_desc(&map_do);
    }
    if (warp == 0) { tmem_alloc(smem_u32(&tmem_base_slot), kTmCols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_base_slot;
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    const uint64_t limit = p.wait_limit_ns;

    constexpr uint32_t idesc_s = umma_idesc_bf16(TILE, TILE, false, false);
    constexpr uint32_t idesc_dq = umma_idesc_bf16(TILE, D_QK, false, true);

    uint32_t ph_q = 0, ph_k[2] = {0, 0}, ph_v = 0, ph_s = 0, ph_acc = 0;
    bool ok = true;

    for (int it = blockIdx.x; it < p.n_items && ok; it += gridDim.x) {
        const GroupItem item = p.items[it];
        const int head = item.head, r0 = item.r0;
        const int32_t* list = p.lists + item.list_off;
        const PairDev first = p.pairs[list[0]];
        const int row = r0 + tid;
        const bool row_valid = row < first.q_len;
        const int last_row = min(r0 + TILE, first.q_len) - 1;

        auto tiles_of = [&](const PairDev& pr) -> int {
            int n_keys = pr.k_len;
            if (p.causal) n_keys = min(n_keys, last_row + pr.off + 1);
            return n_keys > 0 ? (n_keys + TILE - 1) / TILE : 0;
        };
        // iterator over (pair of the chunk, kv tile)
        int li = 0, t = 0, nt = 0;
        PairDev cur = first;
        auto seek = [&]() {          // move to the first pair at or after li that has tiles
            while (li < item.list_len) {
                cur = p.pairs[list[li]];
                nt = tiles_of(cur);
                if (nt > 0) return;
                ++li;
            }
        };
        seek();
        int nli = li, ntile = t;     // lookahead iterator (next tile to prefetch)
        PairDev nxt = cur; int nnt = nt;
        auto advance_next = [&]() {
            ++ntile;
            if (ntile >= nnt) {
                ntile = 0; ++nli;
                while (nli < item.list_len) {
                    nxt = p.pairs[list[nli]];
                    nnt = tiles_of(nxt);
                    if (nnt > 0) break;
                    ++nli;
                }
            }
        };
        auto load_k = [&](const PairDev& pr, int tile, int st) {
            mbar_arrive_expect_tx(bar_k0 + 8 * st, 3 * kBox128);
            for (int c = 0; c < 3; ++c)
                tma_load_3d(smem + kK + st * 3 * kBox128 + c * kBox128, &map_k, bar_k0 + 8 * st,
                            c * 64, head, pr.k_tok0 + tile * TILE);
        };
        auto load_v = [&](const PairDev& pr, int tile) {
            mbar_arrive_expect_tx(bar_v, 2 * kBox128);
            for (int c = 0; c < 2; ++c)
                tma_load_3d(smem + kV + c * kBox128, &map_v, bar_v, c * 64, head,
                            pr.k_tok0 + tile * TILE);
        };

        const bool any = li < item.list_len;
        float lse2 = 0.f, dsum = 0.f;
        if (row_valid) {
            const float l = p.lse[static_cast<int64_t>(head) * p.T + first.q_tok0 + row];
            lse2 = (l == neg_inf()) ? pos_inf() : l * 1.4426950408889634f;
            dsum = p.dsum[static_cast<int64_t>(head) * p.T + first.q_tok0 + row];
        }
        if (tid == 0 && any) {
            mbar_arrive_expect_tx(bar_q, 5 * kBox128);
            for (int c = 0; c < 3; ++c)
                tma_load_3d(smem + kQ + c * kBox128, &map_q, bar_q, c * 64, head, first.q_tok0 + r0);
            for (int c = 0; c < 2; ++c)
                tma_load_3d(smem + kDO + c * kBox128, &map_do, bar_q, c * 64, head, first.q_tok0 + r0);
            load_k(cur, 0, 0);
            load_v(cur, 0);
        }

        int step = 0;
        while (li < item.list_len && ok) {
            const int st = step & 1;
            advance_next();
            const bool has_next = nli < item.list_len;
            if (tid == 0) {
                if (has_next) load_k(nxt, ntile, st ^ 1);
                if (step == 0) ok = mbar_wait(bar_q, ph_q, &abort_flag, limit);
                if (ok) ok = mbar_wait(bar_k0 + 8 * st, ph_k[st], &abort_flag, limit);
                if (ok) ok = mbar_wait(bar_v, ph_v, &abort_flag, limit);
                if (ok) {
                    tc_fence_after_sync();
                    const uint32_t qb = smem + kQ, kb = smem + kK + st * 3 * kBox128;
#pragma unroll
                    for (int kk = 0; kk < D_QK / 16; ++kk) {
                        const uint32_t o = (kk >> 2) * kBox128 + (kk & 3) * 32;
                        umma_ss(tm + kTmS, umma_smem_desc_sw128(qb + o, 16, 1024),
                                umma_smem_desc_sw128(kb + o, 16, 1024), idesc_s, kk > 0);
                    }
                    const uint32_t gb = smem + kDO, vb = smem + kV;
#pragma unroll
                    for (int kk = 0; kk < D_V / 16; ++kk) {
                        const uint32_t o = (kk >> 2) * kBox128 + (kk & 3) * 32;
                        umma_ss(tm + kTmDP, umma_smem_desc_sw128(gb + o, 16, 1024),
                                umma_smem_desc_sw128(vb + o, 16, 1024), idesc_s, kk > 0);
                    }
                    umma_commit(bar_s);
                }
            }
            ph_k[st] ^= 1; ph_v ^= 1;
            __syncwarp();
            ok = mbar_wait(bar_s, ph_s, &abort_flag, limit);
            ph_s ^= 1;
            if (!ok) break;
            tc_fence_after_sync();
            if (tid == 0 && has_next) load_v(nxt, ntile);      // V is single-buffered: dP has read it

            // ---- P and dS on this thread's row -----------------------------------------------
            const int col0 = t * TILE;
            int jmax = cur.k_len - 1;
            if (p.causal) jmax = min(jmax, row + cur.off);
            const int cmax = jmax - col0;
#pragma unroll
            for (int c0 = 0; c0 < TILE; c0 += 32) {
                uint32_t s[32], dp[32], ds[16];
                tmem_ld_x32(tm + kTmS + lane_base + c0, s);
                tmem_ld_x32(tm + kTmDP + lane_base + c0, dp);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                    float p0 = ex2_approx(fmaf(__uint_as_float(s[c]), p.scale_log2, -lse2));
                    float p1 = ex2_approx(fmaf(__uint_as_float(s[c + 1]), p.scale_log2, -lse2));
                    if (c0 + c > cmax) p0 = 0.f;
                    if (c0 + c + 1 > cmax) p1 = 0.f;
                    ds[c >> 1] = pack_bf16x2(p0 * (__uint_as_float(dp[c]) - dsum),
                                             p1 * (__uint_as_float(dp[c + 1]) - dsum));
                }
                tmem_st_x16(tm + kTmDS + lane_base + (c0 >> 1), ds);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            __syncthreads();

            if (tid == 0) {
                tc_fence_after_sync();
                const uint32_t kb = smem + kK + st * 3 * kBox128;
#pragma unroll
                for (int kk = 0; kk < TILE / 16; ++kk)
                    umma_ts(tm + kTmDQ, tm + kTmDS + kk * 8,
                            umma_smem_desc_sw128(kb + kk * 2048, kBox128, 1024), idesc_dq,
                            (step > 0) || (kk > 0));
                umma_commit(bar_acc);
            }
            __syncwarp();
            ok = mbar_wait(bar_acc, ph_acc, &abort_flag, limit);
            ph_acc ^= 1;
            if (!ok) break;
            tc_fence_after_sync();

            // advance the current iterator to where the lookahead already is
            ++step;
            li = nli; t = ntile; cur = nxt; nt = nnt;
        }
        if (any) ph_q ^= 1;
        if (!ok) break;

        // ---- epilogue: dQ * scale -> bf16 -----------------------------------------------------
        {
            __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(p.dq) +
                                 (static_cast<int64_t>(first.q_tok0 + row) * p.h + head) * D_QK;
#pragma unroll
            for (int c = 0; c < D_QK; c += 32) {
                uint32_t v[32];
                if (any) {
                    tmem_ld_x32(tm + kTmDQ + lane_base + c, v);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] = 0u;
                }
                if (row_valid) store_row_bf16(dst + c, v, 32, p.scale);
            }
            tc_fence_before_sync();
            __syncthreads();
            tc_fence_after_sync();
        }
    }

    if (!ok || abort_flag) {
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 50000ull) { }
        if (tid == 0) {
            p.status->detail = blockIdx.x;
            p.status->status = HYDRA_ERR_DEVICE_TIMEOUT;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, kTmCols);
}

__global__ void __launch_bounds__(kThreads, 1)
hydra_bwd_dkv_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do,
                     const BwdParams p)
{
    using namespace dkv;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem = (smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t bars[8];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ float s_lse2[2][SUB];
    __shared__ float s_dsum[2][SUB];

    const int tid = threadIdx.x, warp = tid >> 5;
    const uint32_t bar_kv = smem_u32(&bars[0]);     // K and V tile of the item
    const uint32_t bar_q0 = smem_u32(&bars[1]);     // + 8 * stage: Q and dO sub-tile
    const uint32_t bar_s = smem_u32(&bars[3]);      // S^T and dP^T complete
    const uint32_t bar_acc = smem_u32(&bars[4]);    // dV, dK updates complete

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(bar_kv, 1); mbar_init(bar_q0, 1); mbar_init(bar_q0 + 8, 1);
        mbar_init(bar_s, 1); mbar_init(bar_acc, 1);
        fence_mbar_init();
        tma_prefetch_desc(&map_q); tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v); tma_prefetch_desc(&map_do);
    }
    if (warp == 0) { tmem_alloc(smem_u32(&tmem_base_slot), kTmCols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_base_slot;
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    const uint64_t limit = p.wait_limit_ns;

    constexpr uint32_t idesc_st = umma_idesc_bf16(TILE, SUB, false, false);
    constexpr uint32_t idesc_dv = umma_idesc_bf16(TILE, D_V, false, true);
    constexpr uint32_t idesc_dk = umma_idesc_bf16(TILE, D_QK, false, true);

    uint32_t ph_kv = 0, ph_q[2] = {0, 0}, ph_s = 0, ph_acc = 0;
    bool ok = true;

    for (int it = blockIdx.x; it < p.n_items && ok; it += gridDim.x) {
        const GroupItem item = p.items[it];
        const int head = item.head, r0 = item.r0;
        const int32_t* list = p.lists + item.list_off;
        const PairDev first = p.pairs[list[0]];
        const int krow = r0 + tid;                       // kv row inside the chunk
        const bool row_valid = krow < first.k_len;

        auto first_sub = [&](const PairDev& pr) -> int {
            if (!p.causal) return 0;
            const int i_min = r0 - pr.off;               // first q row that sees kv row r0
            return i_min > 0 ? i_min / SUB : 0;
        };
        auto n_sub = [&](const PairDev& pr) -> int { return (pr.q_len + SUB - 1) / SUB; };

        int li = 0, u = 0, nu = 0;
        PairDev cur = first;
        while (li < item.list_len) {
            cur = p.pairs[list[li]];
            u = first_sub(cur); nu = n_sub(cur);
            if (u < nu) break;
            ++li;
        }
        int nli = li, nsub = u, nnu = nu;
        PairDev nxt = cur;
        auto advance_next = [&]() {
            ++nsub;
            if (nsub >= nnu) {
                ++nli;
                while (nli < item.list_len) {
                    nxt = p.pairs[list[nli]];
                    nsub = first_sub(nxt); nnu = n_sub(nxt);
                    if (nsub < nnu) break;
                    ++nli;
                }
            }
        };
        auto load_q = [&](const PairDev& pr, int sub, int st) {
            mbar_arrive_expect_tx(bar_q0 + 8 * st, 5 * kBox64);
            const int tok = pr.q_tok0 + sub * SUB;
            for (int c = 0; c < 3; ++c)
                tma_load_3d(smem + kQ + st * 3 * kBox64 + c * kBox64, &map_q, bar_q0 + 8 * st, c * 64,
                            head, tok);
            for (int c = 0; c < 2; ++c)
                tma_load_3d(smem + kDO + st * 2 * kBox64 + c * kBox64, &map_do, bar_q0 + 8 * st,
                            c * 64, head, tok);
        };
        auto load_stats = [&](const PairDev& pr, int sub, int st) {
            const int i = sub * SUB + (tid & (SUB - 1));
            const bool v = i < pr.q_len;
            const int64_t idx = static_cast<int64_t>(head) * p.T + pr.q_tok0 + i;
            if (tid < SUB) {
                const float l = v ? p.lse[idx] : neg_inf();
                s_lse2[st][tid] = (l == neg_inf()) ? pos_inf() : l * 1.4426950408889634f;
            } else {
                s_dsum[st][tid - SUB] = v ? p.dsum[idx] : 0.f;
            }
        };

        const bool any = li < item.list_len;
        if (any) {
            if (tid == 0) {
                mbar_arrive_expect_tx(bar_kv, 5 * kBox128);
                for (int c = 0; c < 3; ++c)
                    tma_load_3d(smem + kK + c * kBox128, &map_k, bar_kv, c * 64, head, first.k_tok0 + r0);
                for (int c = 0; c < 2; ++c)
                    tma_load_3d(smem + kV + c * kBox128, &map_v, bar_kv, c * 64, head, first.k_tok0 + r0);
                load_q(cur, u, 0);
            }
            load_stats(cur, u, 0);
        }
        __syncthreads();

        int step = 0;
        while (li < item.list_len && ok) {
            const int st = step & 1;
            advance_next();
            const bool has_next = nli < item.list_len;
            if (has_next) load_stats(nxt, nsub, st ^ 1);   // read after this step's __syncthreads
            if (tid == 0) {
                if (has_next) load_q(nxt, nsub, st ^ 1);
                if (step == 0) ok = mbar_wait(bar_kv, ph_kv, &abort_flag, limit);
                if (ok) ok = mbar_wait(bar_q0 + 8 * st, ph_q[st], &abort_flag, limit);
                if (ok) {
                    tc_fence_after_sync();
                    const uint32_t kb = smem + kK, qb = smem + kQ + st * 3 * kBox64;
#pragma unroll
                    for (int kk = 0; kk < D_QK / 16; ++kk)
                        umma_ss(tm + kTmS,
                                umma_smem_desc_sw128(kb + (kk >> 2) * kBox128 + (kk & 3) * 32, 16, 1024),
                                umma_smem_desc_sw128(qb + (kk >> 2) * kBox64 + (kk & 3) * 32, 16, 1024),
                                idesc_st, kk > 0);
                    const uint32_t vb = smem + kV, gb = smem + kDO + st * 2 * kBox64;
#pragma unroll
                    for (int kk = 0; kk < D_V / 16; ++kk)
                        umma_ss(tm + kTmDP,
                                umma_smem_desc_sw128(vb + (kk >> 2) * kBox128 + (kk & 3) * 32, 16, 1024),
                                umma_smem_desc_sw128(gb + (kk >> 2) * kBox64 + (kk & 3) * 32, 16, 1024),
                                idesc_st, kk > 0);
                    umma_commit(bar_s);
                }
            }
            ph_q[st] ^= 1;
            __syncwarp();
            ok = mbar_wait(bar_s, ph_s, &abort_flag, limit);
            ph_s ^= 1;
            if (!ok) break;
            tc_fence_after_sync();

            // ---- P^T and dS^T on this thread's kv row -----------------------------------------
            // q row i = u*64 + c is visible from kv row krow iff i < q_len and krow <= i + off.
            int c_lo = 0;                                   // first visible column
            if (p.causal) c_lo = max(0, krow - cur.off - u * SUB);
            int c_hi = min(SUB, cur.q_len - u * SUB);       // one past the last valid column
            if (!row_valid) c_hi = 0;
#pragma unroll
            for (int c0 = 0; c0 < SUB; c0 += 32) {
                uint32_t s[32], dp[32], pk[16], ds[16];
                tmem_ld_x32(tm + kTmS + lane_base + c0, s);
                tmem_ld_x32(tm + kTmDP + lane_base + c0, dp);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                    const int ca = c0 + c, cb = c0 + c + 1;
                    float p0 = ex2_approx(fmaf(__uint_as_float(s[c]), p.scale_log2, -s_lse2[st][ca]));
                    float p1 = ex2_approx(fmaf(__uint_as_float(s[c + 1]), p.scale_log2, -s_lse2[st][cb]));
                    if (ca < c_lo || ca >= c_hi) p0 = 0.f;
                    if (cb < c_lo || cb >= c_hi) p1 = 0.f;
                    pk[c >> 1] = pack_bf16x2(p0, p1);
                    ds[c >> 1] = pack_bf16x2(p0 * (__uint_as_float(dp[c]) - s_dsum[st][ca]),
                                             p1 * (__uint_as_float(dp[c + 1]) - s_dsum[st][cb]));
                }
                tmem_st_x16(tm + kTmP + lane_base + (c0 >> 1), pk);
                tmem_st_x16(tm + kTmDS + lane_base + (c0 >> 1), ds);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            __syncthreads();

            if (tid == 0) {
                tc_fence_after_sync();
                const uint32_t gb = smem + kDO + st * 2 * kBox64, qb = smem + kQ + st * 3 * kBox64;
#pragma unroll
                for (int kk = 0; kk < SUB / 16; ++kk)
                    umma_ts(tm + kTmDV, tm + kTmP + kk * 8,
                            umma_smem_desc_sw128(gb + kk * 2048, kBox64, 1024), idesc_dv,
                            (step > 0) || (kk > 0));
#pragma unroll
                for (int kk = 0; kk < SUB / 16; ++kk)
                    umma_ts(tm + kTmDK, tm + kTmDS + kk * 8,
                            umma_smem_desc_sw128(qb + kk * 2048, kBox64, 1024), idesc_dk,
                            (step > 0) || (kk > 0));
                umma_commit(bar_acc);
            }
            __syncwarp();
            ok = mbar_wait(bar_acc, ph_acc, &abort_flag, limit);
            ph_acc ^= 1;
            if (!ok) break;
            tc_fence_after_sync();

            ++step;
            li = nli; u = nsub; cur = nxt; nu = nnu;
        }
        if (any) ph_kv ^= 1;
        if (!ok) break;

        // ---- epilogue: dK * scale, dV -> bf16 ---------------------------------------------------
        {
            const int64_t tok = static_cast<int64_t>(first.k_tok0) + krow;
            __nv_bfloat16* dkp = static_cast<__nv_bfloat16*>(p.dk) + (tok * p.h + head) * D_QK;
            __nv_bfloat16* dvp = static_cast<__nv_bfloat16*>(p.dv) + (tok * p.h + head) * D_V;
#pragma unroll
            for (int c = 0; c < D_QK; c += 32) {
                uint32_t v[32];
                if (any) {
                    tmem_ld_x32(tm + kTmDK + lane_base + c, v);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] = 0u;
                }
                if (row_valid) store_row_bf16(dkp + c, v, 32, p.scale);
            }
#pragma unroll
            for (int c = 0; c < D_V; c += 32) {
                uint32_t v[32];
                if (any) {
                    tmem_ld_x32(tm + kTmDV + lane_base + c, v);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] = 0u;
                }
                if (row_valid) store_row_bf16(dvp + c, v, 32, 1.f);
            }
            tc_fence_before_sync();
            __syncthreads();
            tc_fence_after_sync();
        }
    }

    if (!ok || abort_flag) {
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 50000ull) { }
        if (tid == 0) {
            p.status->detail = blockIdx.x;
            p.status->status = HYDRA_ERR_DEVICE_TIMEOUT;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, kTmCols);
}

cudaError_t launch_bwd_dq(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                          const CUtensorMap& mdo, const BwdParams& p, int grid, cudaStream_t stream)
{
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(hydra_bwd_dq_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(bwd_dq_smem_bytes()));
        if (e != cudaSuccess) return e;
        configured = true;
    }
    hydra_bwd_dq_kernel<<<grid, kThreads, bwd_dq_smem_bytes(), stream>>>(mq, mk, mv, mdo, p);
    return cudaGetLastError();
}

cudaError_t launch_bwd_dkv(const CUtensorMap& mq_sub, const CUtensorMap& mk, const CUtensorMap& mv,
                           const CUtensorMap& mdo_sub, const BwdParams& p, int grid, cudaStream_t stream)
{
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(hydra_bwd_dkv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(bwd_dkv_smem_bytes()));
        if (e != cudaSuccess) return e;
        configured = true;
    }
    hydra_bwd_dkv_kernel<<<grid, kThreads, bwd_dkv_smem_bytes(), stream>>>(mq_sub, mk, mv, mdo_sub, p);
    return cudaGetLastError();
}

}  // namespace hydra
