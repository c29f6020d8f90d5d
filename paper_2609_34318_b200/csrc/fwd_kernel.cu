// Forward attention of (q-chunk, kv-chunk) pairs on sm_100a: TMA -> shared memory -> tcgen05 UMMA
// with S and O accumulated in tensor memory, online softmax on thread-private rows.
//
// One CTA walks a strided share of the work list; a work item is one 128-row q tile of one pair and
// head. Per kv tile: S = Q K^T (SS UMMA, both operands K-major), softmax in the exp2 domain with
// the running row maximum, P written back to tensor memory as packed bf16, O += P V (TS UMMA, V
// read as an MN-major B operand straight from its token-major layout). Thread r of the CTA owns
// row r of the tile = TMEM lane r, so row max and row sum need no cross-thread traffic.
#include <cuda_bf16.h>

#include "hydra_internal.h"
#include "sm100_ptx.cuh"

namespace hydra {

namespace {

constexpr int kThreads = 128;
constexpr uint32_t kBoxBytes = TILE * 128;            // one [128 rows x 64 bf16] swizzled box
constexpr uint32_t kQBytes = 3 * kBoxBytes;           // 128 x 192
constexpr uint32_t kKBytes = 3 * kBoxBytes;
constexpr uint32_t kVBytes = 2 * kBoxBytes;           // 128 x 128
constexpr int kStages = 2;
constexpr uint32_t kSmemQ = 0;
constexpr uint32_t kSmemK = kSmemQ + kQBytes;
constexpr uint32_t kSmemV = kSmemK + kStages * kKBytes;
constexpr uint32_t kSmemTotal = kSmemV + kStages * kVBytes;   // 212,992 B
// TMEM columns
constexpr uint32_t kTmS = 0, kTmO = 128, kTmP = 256, kTmCols = 512;

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

}  // namespace

size_t fwd_smem_bytes() { return kSmemTotal + 1024; }

__global__ void __launch_bounds__(kThreads, 1)
hydra_fwd_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const FwdParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem = (smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t bars[8];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5;
    const uint32_t bar_q = smem_u32(&bars[0]);
    const uint32_t bar_k0 = smem_u32(&bars[1]);   // + 8 * stage
    const uint32_t bar_v0 = smem_u32(&bars[3]);   // + 8 * stage
    const uint32_t bar_s = smem_u32(&bars[5]);
    const uint32_t bar_o = smem_u32(&bars[6]);

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(bar_q, 1);
        mbar_init(bar_k0, 1); mbar_init(bar_k0 + 8, 1);
        mbar_init(bar_v0, 1); mbar_init(bar_v0 + 8, 1);
        mbar_init(bar_s, 1); mbar_init(bar_o, 1);
        fence_mbar_init();
        tma_prefetch_desc(&map_q); tma_prefetch_desc(&map_k); tma_prefetch_desc(&map_v);
    }
    if (warp == 0) { tmem_alloc(smem_u32(&tmem_base_slot), kTmCols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_base_slot;
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    const uint64_t limit = p.wait_limit_ns;

    constexpr uint32_t idesc_s = umma_idesc_bf16(TILE, TILE, false, false);
    constexpr uint32_t idesc_o = umma_idesc_bf16(TILE, D_V, false, true);

    uint32_t ph_q = 0, ph_k[2] = {0, 0}, ph_v[2] = {0, 0}, ph_s = 0, ph_o = 0;
    bool ok = true;

    for (int it = blockIdx.x; it < p.n_items && ok; it += gridDim.x) {
        const FwdItem item = p.items[it];
        const PairDev pr = p.pairs[item.pair];
        const int head = item.head, q0 = item.q0, n_kv = item.n_kv;
        const int row = q0 + tid;                       // q row inside the pair
        const bool row_valid = row < pr.q_len;

        auto load_kv = [&](int j, int st) {
            const int tok = pr.k_tok0 + j * TILE;
            mbar_arrive_expect_tx(bar_k0 + 8 * st, kKBytes);
            for (int c = 0; c < 3; ++c)
                tma_load_3d(smem + kSmemK + st * kKBytes + c * kBoxBytes, &map_k, bar_k0 + 8 * st,
                            c * 64, head, tok);
            mbar_arrive_expect_tx(bar_v0 + 8 * st, kVBytes);
            for (int c = 0; c < 2; ++c)
                tma_load_3d(smem + kSmemV + st * kVBytes + c * kBoxBytes, &map_v, bar_v0 + 8 * st,
                            c * 64, head, tok);
        };

        if (tid == 0 && n_kv > 0) {
            mbar_arrive_expect_tx(bar_q, kQBytes);
            for (int c = 0; c < 3; ++c)
                tma_load_3d(smem + kSmemQ + c * kBoxBytes, &map_q, bar_q, c * 64, head,
                            pr.q_tok0 + q0);
            load_kv(0, 0);
        }

        float m_run = neg_inf(), l_run = 0.f;

        for (int j = 0; j < n_kv && ok; ++j) {
            const int st = j & 1;
            if (tid == 0) {
                if (j + 1 < n_kv) load_kv(j + 1, st ^ 1);
                if (j == 0) ok = mbar_wait(bar_q, ph_q, &abort_flag, limit);
                if (ok) ok = mbar_wait(bar_k0 + 8 * st, ph_k[st], &abort_flag, limit);
                if (ok) {
                    tc_fence_after_sync();
                    const uint32_t qb = smem + kSmemQ, kb = smem + kSmemK + st * kKBytes;
#pragma unroll
                    for (int kk = 0; kk < D_QK / 16; ++kk) {
                        const uint32_t o = (kk >> 2) * kBoxBytes + (kk & 3) * 32;
                        umma_ss(tm + kTmS, umma_smem_desc_sw128(qb + o, 16, 1024),
                                umma_smem_desc_sw128(kb + o, 16, 1024), idesc_s, kk > 0);
                    }
                    umma_commit(bar_s);
                }
            }
            ph_k[st] ^= 1;
            __syncwarp();
            ok = mbar_wait(bar_s, ph_s, &abort_flag, limit);
            ph_s ^= 1;
            if (!ok) break;
            tc_fence_after_sync();

            // ---- softmax on this thread's row -------------------------------------------------
            uint32_t s[TILE];
#pragma unroll
            for (int c = 0; c < TILE; c += 32) tmem_ld_x32(tm + kTmS + lane_base + c, s + c);
            tmem_wait_ld();

            const int col0 = j * TILE;
            const bool need_mask =
                (col0 + TILE > pr.k_len) || (p.causal && (col0 + TILE - 1 > q0 + pr.off));
            if (need_mask) {
                int jmax = pr.k_len - 1;
                if (p.causal) jmax = min(jmax, row + pr.off);
                const int cmax = jmax - col0;          // columns 0..cmax are visible
#pragma unroll
                for (int c = 0; c < TILE; ++c)
                    if (c > cmax) s[c] = __float_as_uint(neg_inf());
            }
            float mx = neg_inf();
#pragma unroll
            for (int c = 0; c < TILE; ++c) mx = fmaxf(mx, __uint_as_float(s[c]));
            const float m_new = fmaxf(m_run, mx * p.scale_log2);
            const float m_use = (m_new == neg_inf()) ? 0.f : m_new;
            const float alpha = ex2_approx(m_run - m_use);
            float rs = 0.f;
            uint32_t pk[TILE / 2];
#pragma unroll
            for (int c = 0; c < TILE; c += 2) {
                const float p0 = ex2_approx(fmaf(__uint_as_float(s[c]), p.scale_log2, -m_use));
                const float p1 = ex2_approx(fmaf(__uint_as_float(s[c + 1]), p.scale_log2, -m_use));
                rs += p0 + p1;
                pk[c >> 1] = pack_bf16x2(p0, p1);
            }
            l_run = l_run * alpha + rs;
            m_run = m_new;
#pragma unroll
            for (int c = 0; c < TILE / 2; c += 32) tmem_st_x32(tm + kTmP + lane_base + c, pk + c);

            // rescale the running O (the previous P V has completed: bar_o was waited on)
            if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
                for (int c = 0; c < D_V; c += 32) {
                    uint32_t o[32];
                    tmem_ld_x32(tm + kTmO + lane_base + c, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                    tmem_st_x32(tm + kTmO + lane_base + c, o);
                }
            }
            tmem_wait_st();
            tc_fence_before_sync();
            __syncthreads();

            if (tid == 0) {
                tc_fence_after_sync();
                ok = mbar_wait(bar_v0 + 8 * st, ph_v[st], &abort_flag, limit);
                if (ok) {
                    tc_fence_after_sync();
                    const uint32_t vb = smem + kSmemV + st * kVBytes;
#pragma unroll
                    for (int kk = 0; kk < TILE / 16; ++kk)
                        umma_ts(tm + kTmO, tm + kTmP + kk * 8,
                                umma_smem_desc_sw128(vb + kk * 2048, kBoxBytes, 1024), idesc_o,
                                (j > 0) || (kk > 0));
                    umma_commit(bar_o);
                }
            }
            ph_v[st] ^= 1;
            __syncwarp();
            ok = mbar_wait(bar_o, ph_o, &abort_flag, limit);
            ph_o ^= 1;
            if (!ok) break;
            tc_fence_after_sync();
        }
        if (n_kv > 0) ph_q ^= 1;
        if (!ok) break;

        // ---- epilogue: O / l -> bf16, LSE = ln2 * (m + log2 l) --------------------------------
        {
            const int64_t rows_total = pr.to_part ? p.part_rows : p.T;
            __nv_bfloat16* obase = static_cast<__nv_bfloat16*>(pr.to_part ? p.o_part : p.out);
            float* lbase = pr.to_part ? p.lse_part : p.lse;
            const int64_t orow = static_cast<int64_t>(pr.out_row0) + row;
            const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
            uint4* dst = reinterpret_cast<uint4*>(obase + (orow * p.h + head) * D_V);
#pragma unroll
            for (int c = 0; c < D_V; c += 32) {
                uint32_t o[32];
                if (n_kv > 0) {
                    tmem_ld_x32(tm + kTmO + lane_base + c, o);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) o[e] = 0u;
                }
                if (row_valid) {
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(o[e + 0]) * inv_l, __uint_as_float(o[e + 1]) * inv_l);
                        w.y = pack_bf16x2(__uint_as_float(o[e + 2]) * inv_l, __uint_as_float(o[e + 3]) * inv_l);
                        w.z = pack_bf16x2(__uint_as_float(o[e + 4]) * inv_l, __uint_as_float(o[e + 5]) * inv_l);
                        w.w = pack_bf16x2(__uint_as_float(o[e + 6]) * inv_l, __uint_as_float(o[e + 7]) * inv_l);
                        dst[(c + e) >> 3] = w;
                    }
                }
            }
            if (row_valid)
                lbase[static_cast<int64_t>(head) * rows_total + orow] =
                    (l_run > 0.f) ? (m_run + __log2f(l_run)) * 0.6931471805599453f : neg_inf();
            tc_fence_before_sync();
            __syncthreads();      // every row has left TMEM before the next item's UMMAs overwrite it
            tc_fence_after_sync();
        }
    }

    if (!ok || abort_flag) {
        // A wait ran out. Give copies still in flight time to land, then report and leave.
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

cudaError_t launch_fwd(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                       const FwdParams& p, int grid, cudaStream_t stream)
{
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(hydra_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(fwd_smem_bytes()));
        if (e != cudaSuccess) return e;
        configured = true;
    }
    hydra_fwd_kernel<<<grid, kThreads, fwd_smem_bytes(), stream>>>(mq, mk, mv, p);
    return cudaGetLastError();
}

}  // namespace hydra
