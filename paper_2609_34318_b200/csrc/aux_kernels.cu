// The bandwidth-bound steps around the tensor-core kernels:
//   hydra_lse_merge_kernel  n-way log-sum-exp merge of the partial (O, LSE) of a q chunk
//   hydra_bwd_prep_kernel   D = rowsum(dO * O)
// Both move every byte once with 16-byte accesses: 16 lanes own one (row, head) vector of 128 bf16.
#include <cuda_bf16.h>

#include "hydra_internal.h"

namespace hydra {

namespace {

constexpr int kThreads = 256;
constexpr int kLanesPerUnit = 16;                 // 16 lanes x 8 bf16 = one 128-wide row
constexpr int kUnitsPerPass = kThreads / kLanesPerUnit;

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

__device__ __forceinline__ void unpack8(const uint4& w, float* f)
{
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&w);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 t = __bfloat1622float2(h[i]);
        f[2 * i] = t.x;
        f[2 * i + 1] = t.y;
    }
}

__device__ __forceinline__ uint4 pack8(const float* f)
{
    uint4 w;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&w);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    return w;
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

}  // namespace

// One block = MERGE_ROWS consecutive rows of one chunk, all heads.  For (row, head):
//   M = max_p LSE_p;  Z = sum_p exp(LSE_p - M);  LSE = M + ln Z;  O = sum_p (exp(LSE_p - M) / Z) O_p
__global__ void __launch_bounds__(kThreads)
hydra_lse_merge_kernel(const MergeParams p)
{
    const MergeItem item = p.items[blockIdx.x];
    const MergeGroup g = p.groups[item.group];
    const int32_t* part_row = p.lists + g.list_off;
    const int rows = min(MERGE_ROWS, g.rows - item.row0);
    const int lane = threadIdx.x & (kLanesPerUnit - 1);
    const int unit0 = threadIdx.x / kLanesPerUnit;
    const uint4* o_part = static_cast<const uint4*>(p.o_part);
    uint4* out = static_cast<uint4*>(p.out);
    constexpr int kVecPerRow = D_V / 8;           // uint4 per (row, head)

    for (int u = unit0; u < rows * p.h; u += kUnitsPerPass) {
        const int r = item.row0 + u / p.h, a = u % p.h;
        float m = neg_inf();
        for (int q = 0; q < g.n_parts; ++q)
            m = fmaxf(m, __ldg(p.lse_part + static_cast<int64_t>(a) * p.part_rows + part_row[q] + r));
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.f;
        float z = 0.f;
        if (m != neg_inf()) {
            for (int q = 0; q < g.n_parts; ++q) {
                const int64_t prow = static_cast<int64_t>(part_row[q]) + r;
                const float w = __expf(__ldg(p.lse_part + static_cast<int64_t>(a) * p.part_rows + prow) - m);
                if (w == 0.f) continue;
                z += w;
                float f[8];
                unpack8(ld_stream(o_part + (prow * p.h + a) * kVecPerRow + lane), f);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = fmaf(w, f[e], acc[e]);
            }
            const float inv = 1.f / z;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] *= inv;
        }
        const int64_t tok = static_cast<int64_t>(g.out_tok0) + r;
        out[(tok * p.h + a) * kVecPerRow + lane] = pack8(acc);
        if (lane == 0)
            p.lse[static_cast<int64_t>(a) * p.T + tok] = (m == neg_inf()) ? neg_inf() : m + __logf(z);
    }
}

// D[a, t] = sum_e dO[t, a, e] * O[t, a, e]
__global__ void __launch_bounds__(kThreads)
hydra_bwd_prep_kernel(const uint4* __restrict__ dout, const uint4* __restrict__ out,
                      float* __restrict__ dsum, int64_t T, int32_t h)
{
    const int lane = threadIdx.x & (kLanesPerUnit - 1);
    const int64_t units = T * h;
    constexpr int kVecPerRow = D_V / 8;
    for (int64_t u = static_cast<int64_t>(blockIdx.x) * kUnitsPerPass + threadIdx.x / kLanesPerUnit;
         u < units; u += static_cast<int64_t>(gridDim.x) * kUnitsPerPass) {
        float a[8], b[8];
        unpack8(ld_stream(dout + u * kVecPerRow + lane), a);
        unpack8(ld_stream(out + u * kVecPerRow + lane), b);
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) s = fmaf(a[e], b[e], s);
#pragma unroll
        for (int o = kLanesPerUnit / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) {
            const int64_t t = u / h;
            const int a_head = static_cast<int>(u % h);
            dsum[static_cast<int64_t>(a_head) * T + t] = s;
        }
    }
}

cudaError_t launch_merge(const MergeParams& p, cudaStream_t stream)
{
    if (p.n_items == 0) return cudaSuccess;
    hydra_lse_merge_kernel<<<p.n_items, kThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_bwd_prep(const void* dout, const void* out, float* dsum, int64_t T, int32_t h,
                            cudaStream_t stream)
{
    if (T * h == 0) return cudaSuccess;
    const int64_t passes = (T * h + kUnitsPerPass - 1) / kUnitsPerPass;
    const int grid = static_cast<int>(passes < 148 * 16 ? passes : 148 * 16);
    hydra_bwd_prep_kernel<<<grid, kThreads, 0, stream>>>(static_cast<const uint4*>(dout),
                                                         static_cast<const uint4*>(out), dsum, T, h);
    return cudaGetLastError();
}

}  // namespace hydra
