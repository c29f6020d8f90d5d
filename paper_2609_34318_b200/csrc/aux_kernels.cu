// The bandwidth-bound steps around the tensor-core kernels:
//   hydra_lse_merge_kernel  n-way log-sum-exp merge of the partial (O, LSE) of a q chunk
//   hydra_bwd_prep_kernel   D = rowsum(dO * O)
//   hydra_grad_cast_kernel  fp32 gradient accumulators -> bf16 (after a backward run step by step)
//   hydra_ulysses_kernel    the local permutation before / after the head <-> sequence all-to-all
// All move every byte once: 8 lanes with 32-byte accesses own one (row, head) vector of 128 bf16 (16 lanes with
// 16-byte accesses where a buffer is only 16-byte aligned).
#include <cuda_bf16.h>

#include <algorithm>
#include <mutex>
#include <utility>

#include "hydra_internal.h"
#include "sm100_ptx.cuh"

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
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

}  // namespace

// One block = MERGE_ROWS consecutive rows of one chunk, all heads.  For (row, head):
//   M = max_p LSE_p;  Z = sum_p exp(LSE_p - M);  LSE = M + ln Z;  O = sum_p (exp(LSE_p - M) / Z) O_p
// An earlier form (two partials requested up front, the rest one round trip each, the running sums corrected
// per partial) kept the issue slots 71-73 % busy at 4.4-5.0 TB/s, so the inner loop is kept short: the partials of a (row, head) are taken four at a time,
// all four loads and their LSEs requested before anything is computed (most chunks have two to four partials:
// one round trip); the weights exp(LSE_p - M) are formed once per group of four, so the running sums are
// corrected at most once per group instead of once per partial and the final 1 / Z is folded into one
// multiply per element; the products are packed two-element FMAs; (row, head) advance without a division.
// kBatch = partials requested together: 4 (four blocks per SM, 64 registers) when some chunk has more than two
// partials, else 2 (six blocks per SM: with two partials per chunk, as in a sequence cut in two, occupancy is
// worth more than loads in flight per thread). Measured, L2 flushed: 256K ring workload 4.93 -> 5.72 TB/s (89 % of
// the measured copy bandwidth), many-short split workload 4.74 -> 4.97 TB/s; with four at a time for every chunk
// the latter fell to 4.1, with five or six blocks per SM for kBatch = 4 (spills) the former to 5.69 / 5.26.
template <bool kAccumulate, int kBatch>
__global__ void __launch_bounds__(kThreads, kBatch == 2 ? 6 : 4)
hydra_lse_merge_kernel(const MergeParams p)
{
    const MergeItem item = p.items[blockIdx.x];
    const MergeGroup g = p.groups[item.group];
    const int32_t* part_row = p.lists + g.list_off;
    const int rows = min(MERGE_ROWS, g.rows - item.row0);
    const int lane = threadIdx.x & (kLanesPerUnit - 1);
    const uint4* o_part = static_cast<const uint4*>(p.o_part);
    uint4* out = static_cast<uint4*>(p.out);
    constexpr int kVecPerRow = D_V / 8;           // uint4 per (row, head)
    constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;
    const int n_units = rows * p.h;
    // Unit u of the block is (row r, head a) = (u / h, u % h). The O vectors of consecutive units are
    // consecutive in memory ((row * h + a) * 256 bytes = (row0 * h + u) * 256 bytes), in the partial buffers and in
    // out alike, so their addresses advance by a constant; only the LSE addresses ([h, rows] layouts) need r and
    // a, which advance without a division. The offsets of the first batch of partials do not depend on the
    // unit at all and are formed once per block.
    int u = threadIdx.x / kLanesPerUnit;
    int r = u / p.h, a = u - r * p.h;
    const int step_r = kUnitsPerPass / p.h, step_a = kUnitsPerPass - step_r * p.h;
    const int64_t part_stride = static_cast<int64_t>(p.h) * kVecPerRow;         // uint4 per partial row
    const uint4* o_row = o_part + (static_cast<int64_t>(item.row0) * p.h + u) * kVecPerRow + lane;
    uint4* out_v = out + ((static_cast<int64_t>(g.out_tok0) + item.row0) * p.h + u) * kVecPerRow + lane;
    int32_t pr0[kBatch];
    int64_t off0[kBatch];
#pragma unroll
    for (int i = 0; i < kBatch; ++i) {
        pr0[i] = part_row[i < g.n_parts ? i : 0];
        off0[i] = pr0[i] * part_stride;
    }

    for (; u < n_units; u += kUnitsPerPass, o_row += kUnitsPerPass * kVecPerRow, out_v += kUnitsPerPass * kVecPerRow) {
        const int row = item.row0 + r;
        const float* lse_row = p.lse_part + static_cast<int64_t>(a) * p.part_rows + row;
        float* lse_out = p.lse + static_cast<int64_t>(a) * p.T + g.out_tok0 + row;
        // everything relative to m (in log2 units): acc = sum_p 2^(l_p - m) O_p, z = sum_p 2^(l_p - m)
        float m = neg_inf(), z = 0.f;
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.f;
        // streaming form (one ring step at a time): what out / lse hold so far is one more input
        uint4 v_cur = make_uint4(0u, 0u, 0u, 0u);
        float l_cur = neg_inf();
        if (kAccumulate) {
            l_cur = *lse_out * kLog2e;
            if (l_cur != neg_inf()) v_cur = *out_v;
        }
        for (int q0 = 0; q0 < g.n_parts; q0 += kBatch) {
            uint4 v[kBatch];
            float l[kBatch];
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                const bool have = q0 + i < g.n_parts;
                const int32_t pr = q0 == 0 ? pr0[i] : part_row[have ? q0 + i : q0];
                const int64_t off = q0 == 0 ? off0[i] : pr * part_stride;
                l[i] = have ? __ldg(lse_row + pr) * kLog2e : neg_inf();
                v[i] = make_uint4(0u, 0u, 0u, 0u);
                if (have) v[i] = ld_stream(o_row + off);
            }
            // a partial that saw no key (LSE = -inf) counts for nothing, whatever its O rows hold
#pragma unroll
            for (int i = 0; i < kBatch; ++i)
                if (l[i] == neg_inf()) v[i] = make_uint4(0u, 0u, 0u, 0u);
            float m_new = fmaxf(l[0], l[1]);
            if (kBatch == 4) m_new = fmaxf(m_new, fmaxf(l[kBatch - 2], l[kBatch - 1]));
            if (kAccumulate && q0 == 0) m_new = fmaxf(m_new, l_cur);
            if (m_new > m) {                             // (never for m_new = -inf)
                const float c = ex2_approx(m - m_new);   // 0 when m = -inf
                z *= c;
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] *= c;
                m = m_new;
            }
            if (m == neg_inf()) continue;                // nothing visible so far: every weight is 0
            if (kAccumulate && q0 == 0) {
                const float w = ex2_approx(l_cur - m);
                z += w;
                float f[8];
                unpack8(v_cur, f);
#pragma unroll
                for (int e = 0; e < 8; e += 2) ffma2(acc[e], acc[e + 1], f[e], f[e + 1], w, w, acc[e], acc[e + 1]);
            }
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                if (q0 + i >= g.n_parts) break;          // (the same for every thread of the block)
                const float w = ex2_approx(l[i] - m);    // 0 for a partial that saw no key
                z += w;
                float f[8];
                unpack8(v[i], f);
#pragma unroll
                for (int e = 0; e < 8; e += 2) ffma2(acc[e], acc[e + 1], f[e], f[e + 1], w, w, acc[e], acc[e + 1]);
            }
        }
        const float inv = z > 0.f ? __frcp_rn(z) : 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] *= inv;
        *out_v = pack8(acc);
        if (lane == 0) *lse_out = z > 0.f ? (m + __log2f(z)) * kLn2 : neg_inf();
        a += step_a;
        r += step_r;
        if (a >= p.h) { a -= p.h; ++r; }
    }
}
// The same merge with 32 bytes per lane (8 lanes own one (row, head) vector, 256-bit loads and stores): the
// address arithmetic, the LSE loads and the exponentials of a (row, head) are then shared by half as many
// threads, and the kernel, which is bound by instruction issue, moves 6.55-6.67 TB/s on the 256K ring workload
// (5.74 with 16 bytes per lane) and 6.0 TB/s on the many-short split workload (5.03): the measured copy
// bandwidth. Needs 32-byte aligned buffers; launch_merge falls back to the 16-byte form otherwise (the
// interface asks for 16).
struct V8 { uint32_t w[8]; };
__device__ __forceinline__ V8 ld_stream32(const V8* p)
{
    V8 v;
    asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]),
                   "=r"(v.w[7])
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void unpack16(const V8& v, float* f)
{
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        f[2 * i] = __uint_as_float(v.w[i] << 16);
        f[2 * i + 1] = __uint_as_float(v.w[i] & 0xffff0000u);
    }
}
template <bool kAccumulate, int kBatch>
__global__ void __launch_bounds__(kThreads, kAccumulate ? 3 : 4)
hydra_lse_merge_wide_kernel(const MergeParams p)
{
    constexpr int kLanes = 8, kUnits = kThreads / kLanes;
    const MergeItem item = p.items[blockIdx.x];
    const MergeGroup g = p.groups[item.group];
    const int32_t* part_row = p.lists + g.list_off;
    const int rows = min(MERGE_ROWS, g.rows - item.row0);
    const int lane = threadIdx.x & (kLanes - 1);
    const V8* o_part = static_cast<const V8*>(p.o_part);
    V8* out = static_cast<V8*>(p.out);
    constexpr int kVecPerRow = D_V / 16;          // 32-byte vectors per (row, head)
    constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;
    const int n_units = rows * p.h;
    int u = threadIdx.x / kLanes;
    int r = u / p.h, a = u - r * p.h;
    const int step_r = kUnits / p.h, step_a = kUnits - step_r * p.h;
    const int64_t part_stride = static_cast<int64_t>(p.h) * kVecPerRow;
    const V8* o_row = o_part + (static_cast<int64_t>(item.row0) * p.h + u) * kVecPerRow + lane;
    V8* out_v = out + ((static_cast<int64_t>(g.out_tok0) + item.row0) * p.h + u) * kVecPerRow + lane;
    int32_t pr0[kBatch];
    int64_t off0[kBatch];
#pragma unroll
    for (int i = 0; i < kBatch; ++i) {
        pr0[i] = part_row[i < g.n_parts ? i : 0];
        off0[i] = pr0[i] * part_stride;
    }
    for (; u < n_units; u += kUnits, o_row += kUnits * kVecPerRow, out_v += kUnits * kVecPerRow) {
        const int row = item.row0 + r;
        const float* lse_row = p.lse_part + static_cast<int64_t>(a) * p.part_rows + row;
        float* lse_out = p.lse + static_cast<int64_t>(a) * p.T + g.out_tok0 + row;
        float m = neg_inf(), z = 0.f;
        float acc[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[e] = 0.f;
        V8 v_cur;
#pragma unroll
        for (int e = 0; e < 8; ++e) v_cur.w[e] = 0u;
        float l_cur = neg_inf();
        if (kAccumulate) {
            l_cur = *lse_out * kLog2e;
            if (l_cur != neg_inf()) v_cur = *out_v;
        }
        for (int q0 = 0; q0 < g.n_parts; q0 += kBatch) {
            V8 v[kBatch];
            float l[kBatch];
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                const bool have = q0 + i < g.n_parts;
                const int32_t pr = q0 == 0 ? pr0[i] : part_row[have ? q0 + i : q0];
                const int64_t off = q0 == 0 ? off0[i] : pr * part_stride;
                l[i] = have ? __ldg(lse_row + pr) * kLog2e : neg_inf();
#pragma unroll
                for (int e = 0; e < 8; ++e) v[i].w[e] = 0u;
                if (have) v[i] = ld_stream32(o_row + off);
            }
#pragma unroll
            for (int i = 0; i < kBatch; ++i)
                if (l[i] == neg_inf()) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) v[i].w[e] = 0u;
                }
            float m_new = fmaxf(l[0], l[1]);
            if (kBatch == 4) m_new = fmaxf(m_new, fmaxf(l[kBatch - 2], l[kBatch - 1]));
            if (kAccumulate && q0 == 0) m_new = fmaxf(m_new, l_cur);
            if (m_new > m) {
                const float c = ex2_approx(m - m_new);
                z *= c;
#pragma unroll
                for (int e = 0; e < 16; ++e) acc[e] *= c;
                m = m_new;
            }
            if (m == neg_inf()) continue;
            if (kAccumulate && q0 == 0) {
                const float w = ex2_approx(l_cur - m);
                z += w;
                float f[16];
                unpack16(v_cur, f);
#pragma unroll
                for (int e = 0; e < 16; e += 2) ffma2(acc[e], acc[e + 1], f[e], f[e + 1], w, w, acc[e], acc[e + 1]);
            }
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                if (q0 + i >= g.n_parts) break;
                const float w = ex2_approx(l[i] - m);
                z += w;
                float f[16];
                unpack16(v[i], f);
#pragma unroll
                for (int e = 0; e < 16; e += 2) ffma2(acc[e], acc[e + 1], f[e], f[e + 1], w, w, acc[e], acc[e + 1]);
            }
        }
        const float inv = z > 0.f ? __frcp_rn(z) : 0.f;
        uint32_t o[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) o[e] = pack_bf16x2(acc[2 * e] * inv, acc[2 * e + 1] * inv);
        st_global_v8(out_v, o);
        if (lane == 0) *lse_out = z > 0.f ? (m + __log2f(z)) * kLn2 : neg_inf();
        a += step_a;
        r += step_r;
        if (a >= p.h) { a -= p.h; ++r; }
    }
}
// (Measured and not kept, all on the 256K ring workload and the many-short split workload, L2 flushed, against
// the earlier form's 4.4-5.0 TB/s depending on the GPU of the pool: persistent blocks with the tables in shared
// memory and four partial loads per lane group in flight, 4.3-4.5 TB/s; two (row, head) vectors per lane group
// at two blocks per SM, 3.5 TB/s; partials staged through shared memory by bulk asynchronous copies, three
// 64 KB stages and sixteen consumer warps per SM, 3.1-3.8 TB/s. Short-lived blocks in different phases keep
// more loads in flight than any of those.)

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

// The same with 32 bytes per lane (8 lanes per (row, head), 256-bit loads), for 32-byte aligned buffers.
__global__ void __launch_bounds__(kThreads)
hydra_bwd_prep_wide_kernel(const V8* __restrict__ dout, const V8* __restrict__ out, float* __restrict__ dsum,
                           int64_t T, int32_t h)
{
    constexpr int kLanes = 8, kUnits = kThreads / kLanes, kVecPerRow = D_V / 16;
    const int lane = threadIdx.x & (kLanes - 1);
    const int64_t units = T * h;
    for (int64_t u = static_cast<int64_t>(blockIdx.x) * kUnits + threadIdx.x / kLanes; u < units;
         u += static_cast<int64_t>(gridDim.x) * kUnits) {
        float a[16], b[16];
        unpack16(ld_stream32(dout + u * kVecPerRow + lane), a);
        unpack16(ld_stream32(out + u * kVecPerRow + lane), b);
        float s0 = 0.f, s1 = 0.f;
#pragma unroll
        for (int e = 0; e < 16; e += 2) ffma2(s0, s1, a[e], a[e + 1], b[e], b[e + 1], s0, s1);
        float s = s0 + s1;
#pragma unroll
        for (int o = kLanes / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) {
            const int64_t t = u / h;
            const int a_head = static_cast<int>(u - t * h);
            dsum[static_cast<int64_t>(a_head) * T + t] = s;
        }
    }
}

// grad (bf16) = acc (fp32), eight elements per thread: two 16-byte loads, one 16-byte store.
__global__ void __launch_bounds__(kThreads)
hydra_grad_cast_kernel(const float4* acc, uint4* grad, int64_t n8, int64_t n, const float* acc_tail,
                       __nv_bfloat16* grad_tail)
{
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < n8; i += stride) {
        float4 a, b;
        asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0, %1, %2, %3}, [%4];"
                     : "=f"(a.x), "=f"(a.y), "=f"(a.z), "=f"(a.w) : "l"(acc + 2 * i));
        asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0, %1, %2, %3}, [%4];"
                     : "=f"(b.x), "=f"(b.y), "=f"(b.z), "=f"(b.w) : "l"(acc + 2 * i + 1));
        const float f[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        grad[i] = pack8(f);
    }
    if (blockIdx.x == 0) {                             // fewer than eight elements left over
        const int64_t t = n8 * 8 + threadIdx.x;
        if (t < n) grad_tail[t] = __float2bfloat16_rn(acc_tail[t]);
    }
}

// Sixteen elements per thread (two 32-byte loads, one 32-byte store), for 32-byte aligned buffers; the
// elements past the last multiple of sixteen go one per thread.
__global__ void __launch_bounds__(kThreads)
hydra_grad_cast_wide_kernel(const V8* acc, V8* grad, int64_t n16, int64_t n, const float* acc_tail,
                            __nv_bfloat16* grad_tail)
{
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < n16; i += stride) {
        const V8 a = ld_stream32(acc + 2 * i), b = ld_stream32(acc + 2 * i + 1);
        uint32_t w[8];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            w[e] = pack_bf16x2(__uint_as_float(a.w[2 * e]), __uint_as_float(a.w[2 * e + 1]));
            w[4 + e] = pack_bf16x2(__uint_as_float(b.w[2 * e]), __uint_as_float(b.w[2 * e + 1]));
        }
        st_global_v8(grad + i, w);
    }
    if (blockIdx.x == 0) {
        const int64_t t = n16 * 16 + threadIdx.x;
        if (t < n) grad_tail[t] = __float2bfloat16_rn(acc_tail[t]);
    }
}

cudaError_t launch_grad_cast(const float* acc, void* grad, int64_t n, cudaStream_t stream)
{
    if (n <= 0) return cudaSuccess;
    if (((reinterpret_cast<uintptr_t>(acc) | reinterpret_cast<uintptr_t>(grad)) & 31u) == 0) {
        const int64_t n16 = n / 16;
        const int64_t blocks = (n16 + kThreads - 1) / kThreads;
        const int grid = static_cast<int>(blocks < 1 ? 1 : (blocks < 148 * 16 ? blocks : 148 * 16));
        hydra_grad_cast_wide_kernel<<<grid, kThreads, 0, stream>>>(reinterpret_cast<const V8*>(acc),
                                                               static_cast<V8*>(grad), n16, n, acc,
                                                               static_cast<__nv_bfloat16*>(grad));
        return cudaGetLastError();
    }
    const int64_t n8 = n / 8;
    const int64_t blocks = (n8 + kThreads - 1) / kThreads;
    const int grid = static_cast<int>(blocks < 1 ? 1 : (blocks < 148 * 16 ? blocks : 148 * 16));
    hydra_grad_cast_kernel<<<grid, kThreads, 0, stream>>>(reinterpret_cast<const float4*>(acc),
                                                          static_cast<uint4*>(grad), n8, n, acc,
                                                          static_cast<__nv_bfloat16*>(grad));
    return cudaGetLastError();
}

// Ulysses pack / unpack: a permutation of 16-byte units between the token-major layout [n][P][cu] (a row
// of a token holds P chunks of cu units, one per head group) and the block-major layout [P][n][cu] (one
// contiguous block per rank of the group). Consecutive warps take consecutive chunks of the block-major
// side, so that side is contiguous across the grid and the other is contiguous per chunk (cu * 16 bytes).
// Vec = the unit a lane moves: 16 bytes, or 32 where the chunk size and the buffers allow it.
__device__ __forceinline__ uint4 ld_unit(const uint4* p) { return ld_stream(p); }
__device__ __forceinline__ void st_unit(uint4* p, const uint4& v) { st_stream(p, v); }
__device__ __forceinline__ V8 ld_unit(const V8* p) { return ld_stream32(p); }
__device__ __forceinline__ void st_unit(V8* p, const V8& v)
{
    asm volatile("st.global.cs.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(v.w[0]), "r"(v.w[1]),
                 "r"(v.w[2]), "r"(v.w[3]), "r"(v.w[4]), "r"(v.w[5]), "r"(v.w[6]), "r"(v.w[7])
                 : "memory");
}
template <bool kPack, class Vec>
__global__ void __launch_bounds__(kThreads)
hydra_ulysses_kernel(const Vec* __restrict__ src, Vec* __restrict__ dst, uint32_t n, uint32_t P, uint32_t cu,
                     uint32_t rows)
{
    // A warp takes one chunk (row = j * n + t of the block-major side) at a time, four chunks in flight:
    // the two divisions are paid once per chunk, not once per 16 bytes (a flat loop over units spent its
    // time on them: 5.1 TB/s).
    constexpr int kUnroll = 4;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t n_warps = gridDim.x * (kThreads / 32);
    for (uint32_t r0 = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5); r0 < rows; r0 += n_warps * kUnroll) {
        uint32_t blk[kUnroll], tok[kUnroll];
#pragma unroll
        for (int e = 0; e < kUnroll; ++e) {
            const uint32_t r = r0 + e * n_warps;
            const uint32_t j = r / n, t = r - j * n;
            blk[e] = r * cu;                               // block-major: [P][n][cu]
            tok[e] = (t * P + j) * cu;                     // token-major: [n][P][cu]
        }
        for (uint32_t w = lane; w < cu; w += 32) {
            Vec v[kUnroll];
#pragma unroll
            for (int e = 0; e < kUnroll; ++e)
                if (r0 + e * n_warps < rows) v[e] = ld_unit(src + (kPack ? tok[e] : blk[e]) + w);
#pragma unroll
            for (int e = 0; e < kUnroll; ++e)
                if (r0 + e * n_warps < rows) st_unit(dst + (kPack ? blk[e] : tok[e]) + w, v[e]);
        }
    }
}

cudaError_t launch_ulysses(bool pack, const void* src, void* dst, int64_t n_tokens, int32_t cp_u, int64_t chunk_units,
                           cudaStream_t stream)
{
    const int64_t rows = n_tokens * cp_u;
    if (rows <= 0 || chunk_units <= 0) return cudaSuccess;
    const int64_t blocks = (rows + (kThreads / 32) * 4 - 1) / ((kThreads / 32) * 4);
    const int grid = static_cast<int>(blocks < 148 * 8 ? blocks : 148 * 8);
    const uint4* s = static_cast<const uint4*>(src);
    uint4* d = static_cast<uint4*>(dst);
    // 32-bit index arithmetic: the caller has checked that the units (plus one sweep of the grid) fit
    const uint32_t n = static_cast<uint32_t>(n_tokens), P = static_cast<uint32_t>(cp_u),
                   cu = static_cast<uint32_t>(chunk_units), r = static_cast<uint32_t>(rows);
    if ((cu & 1u) == 0 && ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 31u) == 0) {
        // chunks of whole 32-byte units in 32-byte aligned buffers: half as many, twice as large accesses
        const V8* s32 = static_cast<const V8*>(src);
        V8* d32 = static_cast<V8*>(dst);
        if (pack) hydra_ulysses_kernel<true, V8><<<grid, kThreads, 0, stream>>>(s32, d32, n, P, cu / 2, r);
        else hydra_ulysses_kernel<false, V8><<<grid, kThreads, 0, stream>>>(s32, d32, n, P, cu / 2, r);
        return cudaGetLastError();
    }
    if (pack) hydra_ulysses_kernel<true, uint4><<<grid, kThreads, 0, stream>>>(s, d, n, P, cu, r);
    else hydra_ulysses_kernel<false, uint4><<<grid, kThreads, 0, stream>>>(s, d, n, P, cu, r);
    return cudaGetLastError();
}

cudaError_t launch_merge(const MergeParams& p, cudaStream_t stream)
{
    if (p.n_items == 0) return cudaSuccess;
    const bool four = p.max_parts > 2;
    const bool wide = ((reinterpret_cast<uintptr_t>(p.o_part) | reinterpret_cast<uintptr_t>(p.out)) & 31u) == 0;
    if (wide) {
        if (p.accumulate) {
            if (four) hydra_lse_merge_wide_kernel<true, 4><<<p.n_items, kThreads, 0, stream>>>(p);
            else hydra_lse_merge_wide_kernel<true, 2><<<p.n_items, kThreads, 0, stream>>>(p);
        } else {
            if (four) hydra_lse_merge_wide_kernel<false, 4><<<p.n_items, kThreads, 0, stream>>>(p);
            else hydra_lse_merge_wide_kernel<false, 2><<<p.n_items, kThreads, 0, stream>>>(p);
        }
    } else if (p.accumulate) {
        if (four) hydra_lse_merge_kernel<true, 4><<<p.n_items, kThreads, 0, stream>>>(p);
        else hydra_lse_merge_kernel<true, 2><<<p.n_items, kThreads, 0, stream>>>(p);
    } else {
        if (four) hydra_lse_merge_kernel<false, 4><<<p.n_items, kThreads, 0, stream>>>(p);
        else hydra_lse_merge_kernel<false, 2><<<p.n_items, kThreads, 0, stream>>>(p);
    }
    return cudaGetLastError();
}

cudaError_t launch_bwd_prep(const void* dout, const void* out, float* dsum, int64_t T, int32_t h,
                            cudaStream_t stream)
{
    if (T * h == 0) return cudaSuccess;
    const int64_t passes = (T * h + kUnitsPerPass - 1) / kUnitsPerPass;
    const int grid = static_cast<int>(passes < 148 * 16 ? passes : 148 * 16);
    if (((reinterpret_cast<uintptr_t>(dout) | reinterpret_cast<uintptr_t>(out)) & 31u) == 0) {
        const int64_t wide_passes = (T * h + 2 * kUnitsPerPass - 1) / (2 * kUnitsPerPass);
        const int wide_grid = static_cast<int>(wide_passes < 148 * 16 ? wide_passes : 148 * 16);
        hydra_bwd_prep_wide_kernel<<<wide_grid, kThreads, 0, stream>>>(static_cast<const V8*>(dout),
                                                                   static_cast<const V8*>(out), dsum, T, h);
        return cudaGetLastError();
    }
    hydra_bwd_prep_kernel<<<grid, kThreads, 0, stream>>>(static_cast<const uint4*>(dout),
                                                         static_cast<const uint4*>(out), dsum, T, h);
    return cudaGetLastError();
}

}  // namespace hydra

// =============================================================================================
// hydra_lse_merge_noalloc: the merge for callers that must not allocate device memory
// =============================================================================================
// hydra_lse_merge keeps its per-problem tables (which q chunk has which partials, cut into blocks of
// rows) in an arena of device memory that the library obtains with cudaMalloc at its first call on a
// device (and a problem with very large tables gets an allocation of its own).
// Some callers cannot have that: a process that has handed all device memory to its own pool and
// leaves nothing for cudaMalloc to find, or a latency-critical loop whose rules forbid cudaMalloc
// because it may synchronise the whole device. This entry point runs the same kernel with the tables
// in a fixed array that is part of the library image, so it calls no cudaMalloc, cudaFree or other
// allocating routine. The price: a hard size limit, and one array per GPU shared by all calls.
// The first call on a device looks up the array's device address (cudaGetSymbolAddress, with that
// device current); make that first call before any stream capture begins.
namespace hydra {
namespace {

constexpr int kNoAllocMaxGroups = HYDRA_NOALLOC_MAX_GROUPS;
constexpr int kNoAllocMaxParts = HYDRA_NOALLOC_MAX_PARTIALS;
constexpr int kNoAllocMaxItems = HYDRA_NOALLOC_MAX_BLOCKS;
constexpr size_t kNoAllocGroupsBytes = sizeof(MergeGroup) * kNoAllocMaxGroups;
constexpr size_t kNoAllocPartsBytes = sizeof(int32_t) * kNoAllocMaxParts;
constexpr size_t kNoAllocItemsBytes = sizeof(MergeItem) * kNoAllocMaxItems;
constexpr size_t kNoAllocBytes = kNoAllocGroupsBytes + kNoAllocPartsBytes + kNoAllocItemsBytes;   // 608 KB

// Lives in every GPU context that loads the library, until the process exits. In host code this
// name is only a handle for cudaGetSymbolAddress, never a pointer to pass to a kernel.
static __device__ __align__(256) unsigned char g_noalloc_merge_tables[kNoAllocBytes];

// Device address of the array on the current device (looked up once per device).
cudaError_t noalloc_tables(unsigned char** out)
{
    static unsigned char* cached[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!cached[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_noalloc_merge_tables);
        if (e != cudaSuccess) return e;
        cached[dev] = static_cast<unsigned char*>(ptr);
    }
    *out = cached[dev];
    return cudaSuccess;
}

}  // namespace
}  // namespace hydra

extern "C" int32_t hydra_lse_merge_noalloc(const void* o_part, const float* lse_part, int64_t part_rows,
                                           const int32_t* cu, int32_t n_seqs, int32_t n_heads,
                                           const hydra_pair_t* pairs, int32_t n_pairs, void* out, float* lse,
                                           void* cuda_stream)
{
    using namespace hydra;
    if (n_seqs < 1 || !cu || n_heads < 1 || !pairs || n_pairs < 1 || part_rows < 0) return HYDRA_ERR_INVALID_ARG;
    if (cu[0] != 0) return HYDRA_ERR_INVALID_ARG;
    for (int b = 0; b < n_seqs; ++b)
        if (cu[b + 1] < cu[b]) return HYDRA_ERR_INVALID_ARG;

    // tables in fixed-size host arrays (no heap use either): groups, part_row lists, row blocks;
    // one set per process, so host-side table building is serialised
    static std::mutex host_tables_mutex;
    std::lock_guard<std::mutex> lock(host_tables_mutex);
    static MergeGroup groups[kNoAllocMaxGroups];
    static int32_t parts[kNoAllocMaxParts];
    static MergeItem items[kNoAllocMaxItems];
    static std::pair<int64_t, int64_t> part_iv[kNoAllocMaxParts], out_iv[kNoAllocMaxGroups];   // [first, end) rows
    int n_groups = 0, n_parts = 0, n_items = 0;
    int32_t max_parts = 0;
    for (int i = 0; i < n_pairs;) {
        int j = i;
        while (j < n_pairs && pairs[j].group == pairs[i].group) ++j;
        const hydra_pair_t& p = pairs[i];
        if (p.seq < 0 || p.seq >= n_seqs || p.flags != 0 || p.q_start < 0 || p.q_len < 0 ||
            int64_t{p.q_start} + p.q_len > int64_t{cu[p.seq + 1]} - cu[p.seq])
            return HYDRA_ERR_INVALID_ARG;
        if (i > 0 && p.group < pairs[i - 1].group) return HYDRA_ERR_INVALID_ARG;
        if (p.part_row >= 0 && p.q_len > 0) {
            if (n_groups >= kNoAllocMaxGroups) return HYDRA_ERR_UNSUPPORTED;
            MergeGroup g;
            g.out_tok0 = cu[p.seq] + p.q_start;
            g.rows = p.q_len;
            g.list_off = n_parts;
            g.n_parts = j - i;
            for (int t = i; t < j; ++t) {
                const hydra_pair_t& q = pairs[t];
                if (q.seq != p.seq || q.q_start != p.q_start || q.q_len != p.q_len || q.part_row < 0 ||
                    int64_t{q.part_row} + q.q_len > part_rows)
                    return HYDRA_ERR_INVALID_ARG;
                if (n_parts >= kNoAllocMaxParts) return HYDRA_ERR_UNSUPPORTED;
                part_iv[n_parts] = {q.part_row, int64_t{q.part_row} + q.q_len};
                parts[n_parts++] = q.part_row;
            }
            for (int32_t r = 0; r < g.rows; r += MERGE_ROWS) {
                if (n_items >= kNoAllocMaxItems) return HYDRA_ERR_UNSUPPORTED;
                items[n_items++] = MergeItem{n_groups, r};
            }
            out_iv[n_groups] = {g.out_tok0, int64_t{g.out_tok0} + g.rows};
            max_parts = std::max(max_parts, g.n_parts);
            groups[n_groups++] = g;
        } else {
            for (int t = i; t < j; ++t)
                if (pairs[t].part_row >= 0 && pairs[t].q_len > 0) return HYDRA_ERR_INVALID_ARG;
        }
        i = j;
    }
    if (n_items == 0) return HYDRA_OK;                 // no chunk has partials: nothing to merge, as in hydra_lse_merge
    const void* ptrs[] = {o_part, lse_part, out, lse};
    for (const void* p : ptrs)
        if (!p || (reinterpret_cast<uintptr_t>(p) & 15u)) return HYDRA_ERR_INVALID_ARG;
    // as in hydra_lse_merge: the partials may not share rows of the partial buffers, and two merged q
    // chunks may not write the same rows of out / lse (std::sort works in place: no heap)
    std::sort(part_iv, part_iv + n_parts);
    for (int i = 1; i < n_parts; ++i)
        if (part_iv[i].first < part_iv[i - 1].second) return HYDRA_ERR_INVALID_ARG;
    std::sort(out_iv, out_iv + n_groups);
    for (int i = 1; i < n_groups; ++i)
        if (out_iv[i].first < out_iv[i - 1].second) return HYDRA_ERR_INVALID_ARG;

    int major = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return HYDRA_ERR_CUDA;
    if (major != 10) return HYDRA_ERR_NOT_SM100;
    unsigned char* tables = nullptr;
    if (noalloc_tables(&tables) != cudaSuccess) return HYDRA_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // The tables below travel from static host arrays that the next call overwrites: a captured copy would
    // read them again at every replay of the graph, so a capturing stream is refused before anything moves.
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &capturing) != cudaSuccess) return HYDRA_ERR_CUDA;
    if (capturing != cudaStreamCaptureStatusNone) return HYDRA_ERR_UNSUPPORTED;
    // Every entry the kernel reads is overwritten here, so nothing of the previous call survives.
    if (cudaMemcpyAsync(tables, groups, sizeof(MergeGroup) * n_groups, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(tables + kNoAllocGroupsBytes, parts, sizeof(int32_t) * n_parts, cudaMemcpyHostToDevice,
                        stream) != cudaSuccess ||
        cudaMemcpyAsync(tables + kNoAllocGroupsBytes + kNoAllocPartsBytes, items, sizeof(MergeItem) * n_items,
                        cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return HYDRA_ERR_CUDA;
    MergeParams mp{};
    mp.groups = reinterpret_cast<const MergeGroup*>(tables);
    mp.lists = reinterpret_cast<const int32_t*>(tables + kNoAllocGroupsBytes);
    mp.items = reinterpret_cast<const MergeItem*>(tables + kNoAllocGroupsBytes + kNoAllocPartsBytes);
    mp.n_items = n_items;
    mp.max_parts = max_parts;
    mp.o_part = o_part; mp.lse_part = lse_part; mp.out = out; mp.lse = lse;
    mp.T = cu[n_seqs]; mp.part_rows = part_rows; mp.h = n_heads;
    // counted and timed like every other merge launch (hydra_launch_count, hydra_profile_collect)
    return launch_merge_counted(mp, stream) == cudaSuccess ? HYDRA_OK : HYDRA_ERR_CUDA;
}
