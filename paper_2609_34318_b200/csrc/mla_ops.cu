// The elementwise steps of a gated multi-head-latent attention block around the attention kernel
// (Section 5.2, "Exposed All-to-All Overlap": the query's rotary embedding; the split of the KV
// up-projection's output into the value and the key's position-free part; the key's rotary embedding and
// concatenation; the output gate), forward and backward. All are bound by HBM: every byte moves once, with
// 16-byte or 4-byte accesses that are contiguous per warp. The paper names the steps, not their formulas;
// the readings taken (rotary pairs (2i, 2i+1), angle = position * theta^(-2i/rope_dim); one rotary key
// vector per token shared by all heads; up-projection rows laid out [key part | value]; gate = sigmoid)
// are stated with each entry point in the header.
#include <cuda_bf16.h>

#include <initializer_list>

#include <cmath>

#include "hydra_internal.h"
#include "sm100_ptx.cuh"

namespace hydra {
namespace {

constexpr int kRopeThreads = 128;
constexpr int kMaxRopePairs = 128;          // rotary dimensions up to 256

__device__ __forceinline__ float2 bf2_to_f2(uint32_t w)
{
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ uint32_t f2_to_bf2(float lo, float hi)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}

// cos / sin of position * theta^(-2i/rope_dim), i < rope_dim / 2, for one token, into shared memory. The
// angle is formed and reduced modulo 2 pi in double precision: at position 262143 a single-precision
// product is off by hundredths of a radian.
__device__ __forceinline__ void rope_table(float* s_cos, float* s_sin, int32_t pos, int32_t rope_dim, double log_theta,
                                           int inverse)
{
    for (int i = threadIdx.x; i < rope_dim / 2; i += blockDim.x) {
        const double freq = exp(-log_theta * (2.0 * i) / rope_dim);
        double ang = static_cast<double>(pos) * freq;
        ang -= 6.283185307179586476925 * floor(ang / 6.283185307179586476925);
        float sn, cs;
        sincosf(static_cast<float>(ang), &sn, &cs);
        s_cos[i] = cs;
        s_sin[i] = inverse ? -sn : sn;
    }
}

// y[t, a, :] = x[t, a, :] with the pairs (2i, 2i+1) of columns [rope_offset, rope_offset + rope_dim) rotated
// by the token's angles. One block per token (grid-stride), the heads' rows as 4-byte pairs.
__global__ void __launch_bounds__(kRopeThreads)
hydra_rope_kernel(const uint32_t* __restrict__ x, const int32_t* __restrict__ positions, uint32_t* __restrict__ y,
                  int64_t n_tokens, int32_t n_heads, int32_t head_dim, int32_t rope_offset, int32_t rope_dim,
                  double log_theta, int inverse, int in_place)
{
    __shared__ float s_cos[kMaxRopePairs], s_sin[kMaxRopePairs];
    const int pairs_per_head = head_dim / 2, p0 = rope_offset / 2, p1 = (rope_offset + rope_dim) / 2;
    for (int64_t t = blockIdx.x; t < n_tokens; t += gridDim.x) {
        __syncthreads();                               // the previous token's table is no longer read
        rope_table(s_cos, s_sin, positions[t], rope_dim, log_theta, inverse);
        __syncthreads();
        const int64_t row0 = t * n_heads * pairs_per_head;
        if (in_place) {                                // only the rotary columns move
            const int n = n_heads * (p1 - p0);
            for (int e = threadIdx.x; e < n; e += kRopeThreads) {
                const int a = e / (p1 - p0), i = e - a * (p1 - p0);
                const int64_t idx = row0 + static_cast<int64_t>(a) * pairs_per_head + p0 + i;
                const float2 v = bf2_to_f2(x[idx]);
                y[idx] = f2_to_bf2(v.x * s_cos[i] - v.y * s_sin[i], v.x * s_sin[i] + v.y * s_cos[i]);
            }
        } else {
            const int n = n_heads * pairs_per_head;
            for (int e = threadIdx.x; e < n; e += kRopeThreads) {
                const int c = e % pairs_per_head;
                uint32_t w = x[row0 + e];
                if (c >= p0 && c < p1) {
                    const float2 v = bf2_to_f2(w);
                    const int i = c - p0;
                    w = f2_to_bf2(v.x * s_cos[i] - v.y * s_sin[i], v.x * s_sin[i] + v.y * s_cos[i]);
                }
                y[row0 + e] = w;
            }
        }
    }
}

// k[t, a, :] = [kv_up[t, a, 0:nope] | rope(k_pe[t, :])], v[t, a, :] = kv_up[t, a, nope:nope+dv]
__global__ void __launch_bounds__(kRopeThreads)
hydra_mla_kv_assemble_kernel(const uint32_t* __restrict__ kv_up, const uint32_t* __restrict__ k_pe,
                             const int32_t* __restrict__ positions, uint32_t* __restrict__ k, uint32_t* __restrict__ v,
                             int64_t n_tokens, int32_t n_heads, int32_t nope, int32_t rope_dim, int32_t dv,
                             double log_theta)
{
    __shared__ float s_cos[kMaxRopePairs], s_sin[kMaxRopePairs];
    __shared__ uint32_t s_pe[kMaxRopePairs];
    const int np = nope / 2, rp = rope_dim / 2, vp = dv / 2;
    const int up_pairs = np + vp, k_pairs = np + rp;
    for (int64_t t = blockIdx.x; t < n_tokens; t += gridDim.x) {
        __syncthreads();
        rope_table(s_cos, s_sin, positions[t], rope_dim, log_theta, 0);
        __syncthreads();
        for (int i = threadIdx.x; i < rp; i += kRopeThreads) {
            const float2 w = bf2_to_f2(k_pe[t * rp + i]);
            s_pe[i] = f2_to_bf2(w.x * s_cos[i] - w.y * s_sin[i], w.x * s_sin[i] + w.y * s_cos[i]);
        }
        __syncthreads();
        const int64_t up0 = t * n_heads * up_pairs, k0 = t * n_heads * k_pairs, v0 = t * n_heads * vp;
        for (int e = threadIdx.x; e < n_heads * up_pairs; e += kRopeThreads) {
            const int a = e / up_pairs, c = e - a * up_pairs;
            const uint32_t w = kv_up[up0 + e];
            if (c < np) k[k0 + static_cast<int64_t>(a) * k_pairs + c] = w;
            else v[v0 + static_cast<int64_t>(a) * vp + (c - np)] = w;
        }
        for (int e = threadIdx.x; e < n_heads * rp; e += kRopeThreads) {
            const int a = e / rp, i = e - a * rp;
            k[k0 + static_cast<int64_t>(a) * k_pairs + np + i] = s_pe[i];
        }
    }
}

// The adjoint: dkv_up[t, a, :] = [dk[t, a, 0:nope] | dv[t, a, :]],
// dk_pe[t, :] = rope^-1( sum_a dk[t, a, nope:nope+rope_dim] ) (summed in fp32, rounded once).
__global__ void __launch_bounds__(kRopeThreads)
hydra_mla_kv_assemble_bwd_kernel(const uint32_t* __restrict__ dk, const uint32_t* __restrict__ dv,
                                 const int32_t* __restrict__ positions, uint32_t* __restrict__ dkv_up,
                                 uint32_t* __restrict__ dk_pe, int64_t n_tokens, int32_t n_heads, int32_t nope,
                                 int32_t rope_dim, int32_t dvd, double log_theta)
{
    __shared__ float s_cos[kMaxRopePairs], s_sin[kMaxRopePairs];
    const int np = nope / 2, rp = rope_dim / 2, vp = dvd / 2;
    const int up_pairs = np + vp, k_pairs = np + rp;
    for (int64_t t = blockIdx.x; t < n_tokens; t += gridDim.x) {
        __syncthreads();
        rope_table(s_cos, s_sin, positions[t], rope_dim, log_theta, 1);
        __syncthreads();
        const int64_t up0 = t * n_heads * up_pairs, k0 = t * n_heads * k_pairs, v0 = t * n_heads * vp;
        for (int e = threadIdx.x; e < n_heads * up_pairs; e += kRopeThreads) {
            const int a = e / up_pairs, c = e - a * up_pairs;
            dkv_up[up0 + e] = c < np ? dk[k0 + static_cast<int64_t>(a) * k_pairs + c]
                                     : dv[v0 + static_cast<int64_t>(a) * vp + (c - np)];
        }
        for (int i = threadIdx.x; i < rp; i += kRopeThreads) {
            float sx = 0.f, sy = 0.f;
            for (int a = 0; a < n_heads; ++a) {
                const float2 w = bf2_to_f2(dk[k0 + static_cast<int64_t>(a) * k_pairs + np + i]);
                sx += w.x;
                sy += w.y;
            }
            dk_pe[t * rp + i] = f2_to_bf2(sx * s_cos[i] - sy * s_sin[i], sx * s_sin[i] + sy * s_cos[i]);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// 16-byte forms of the three kernels above (8 bf16 = 4 rotary pairs per access), used when the head
// dimensions are multiples of 8 and the buffers 16-byte aligned: with 4-byte accesses a thread has 4 bytes
// in flight (key / value assembly 2.0 TB/s on 262 144 tokens x 16 heads, 5.9 with a vector per thread), and the
// pair's frequency is formed once per thread instead of once per token. Flat loops over a token's vectors with
// one integer division per vector: a (head, column) assignment made once per thread and a float reciprocal were
// both measured and are slower (4.5 TB/s).
// ---------------------------------------------------------------------------------------------
// cos / sin table of one token with the pair's frequency already in a register (one pair per thread)
__device__ __forceinline__ void rope_table_fast(float* s_cos, float* s_sin, int32_t pos, int pairs, double freq,
                                                int inverse)
{
    if (static_cast<int>(threadIdx.x) < pairs) {
        double ang = static_cast<double>(pos) * freq;
        ang -= 6.283185307179586476925 * floor(ang / 6.283185307179586476925);
        float sn, cs;
        sincosf(static_cast<float>(ang), &sn, &cs);
        s_cos[threadIdx.x] = cs;
        s_sin[threadIdx.x] = inverse ? -sn : sn;
    }
}
__device__ __forceinline__ uint4 rotate_vec(const uint4& w, const float* cp, const float* sp)
{
    const float4 c4 = *reinterpret_cast<const float4*>(cp), s4 = *reinterpret_cast<const float4*>(sp);
    const float c[4] = {c4.x, c4.y, c4.z, c4.w}, sn[4] = {s4.x, s4.y, s4.z, s4.w};
    const uint32_t in[4] = {w.x, w.y, w.z, w.w};
    uint32_t out[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float2 v = bf2_to_f2(in[j]);
        out[j] = f2_to_bf2(v.x * c[j] - v.y * sn[j], v.x * sn[j] + v.y * c[j]);
    }
    return make_uint4(out[0], out[1], out[2], out[3]);
}

__global__ void __launch_bounds__(kRopeThreads)
hydra_rope_vec_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ positions, uint4* __restrict__ y,
                      int64_t n_tokens, int32_t n_heads, int32_t head_dim, int32_t rope_offset, int32_t rope_dim,
                      double log_theta, int inverse, int in_place)
{
    __shared__ __align__(16) float s_cos[kMaxRopePairs], s_sin[kMaxRopePairs];
    const int vph = head_dim / 8, v0 = rope_offset / 8, nv = rope_dim / 8;
    const double freq = exp(-log_theta * (2.0 * threadIdx.x) / rope_dim);
    for (int64_t t = blockIdx.x; t < n_tokens; t += gridDim.x) {
        __syncthreads();                               // the previous token's table is no longer read
        rope_table_fast(s_cos, s_sin, positions[t], rope_dim / 2, freq, inverse);
        __syncthreads();
        const int64_t row0 = t * n_heads * vph;
        if (in_place) {                                // only the rotary columns move
            for (int e = threadIdx.x; e < n_heads * nv; e += kRopeThreads) {
                const int a = e / nv, i = e - a * nv;
                const int64_t idx = row0 + static_cast<int64_t>(a) * vph + v0 + i;
                y[idx] = rotate_vec(x[idx], s_cos + 4 * i, s_sin + 4 * i);
            }
        } else {
            // the rotary vectors and the others in loops of their own: no lane waits for a rotation it does not
            // do (one loop with a branch per vector: 4.4 instead of 5.65 TB/s)
            const int n_copy = vph - nv;
            for (int e = threadIdx.x; e < n_heads * nv; e += kRopeThreads) {
                const int a = e / nv, i = e - a * nv;
                const int64_t idx = row0 + static_cast<int64_t>(a) * vph + v0 + i;
                y[idx] = rotate_vec(x[idx], s_cos + 4 * i, s_sin + 4 * i);
            }
            for (int e = threadIdx.x; e < n_heads * n_copy; e += kRopeThreads) {
                const int a = e / n_copy, j = e - a * n_copy;
                const int64_t idx = row0 + static_cast<int64_t>(a) * vph + (j < v0 ? j : j + nv);
                y[idx] = x[idx];
            }
        }
    }
}

__global__ void __launch_bounds__(kRopeThreads)
hydra_mla_kv_assemble_vec_kernel(const uint4* __restrict__ kv_up, const uint4* __restrict__ k_pe,
                                 const int32_t* __restrict__ positions, uint4* __restrict__ k, uint4* __restrict__ v,
                                 int64_t n_tokens, int32_t n_heads, int32_t nope, int32_t rope_dim, int32_t dv,
                                 double log_theta)
{
    __shared__ __align__(16) float s_cos[kMaxRopePairs], s_sin[kMaxRopePairs];
    __shared__ uint4 s_pe[kMaxRopePairs / 4];
    const int nv = nope / 8, rv = rope_dim / 8, vv = dv / 8;
    const int up_vecs = nv + vv, k_vecs = nv + rv;
    const double freq = exp(-log_theta * (2.0 * threadIdx.x) / rope_dim);
    for (int64_t t = blockIdx.x; t < n_tokens; t += gridDim.x) {
        __syncthreads();
        rope_table_fast(s_cos, s_sin, positions[t], rope_dim / 2, freq, 0);
        __syncthreads();
        if (static_cast<int>(threadIdx.x) < rv)
            s_pe[threadIdx.x] = rotate_vec(k_pe[t * rv + threadIdx.x], s_cos + 4 * threadIdx.x, s_sin + 4 * threadIdx.x);
        __syncthreads();
        const int64_t up0 = t * n_heads * up_vecs, k0 = t * n_heads * k_vecs, v0 = t * n_heads * vv;
        for (int e = threadIdx.x; e < n_heads * up_vecs; e += kRopeThreads) {
            const int a = e / up_vecs, c = e - a * up_vecs;
            const uint4 w = kv_up[up0 + e];
            if (c < nv) k[k0 + static_cast<int64_t>(a) * k_vecs + c] = w;
            else v[v0 + static_cast<int64_t>(a) * vv + (c - nv)] = w;
        }
        for (int e = threadIdx.x; e < n_heads * rv; e += kRopeThreads) {
            const int a = e / rv, i = e - a * rv;
            k[k0 + static_cast<int64_t>(a) * k_vecs + nv + i] = s_pe[i];
        }
    }
}

__global__ void __launch_bounds__(kRopeThreads)
hydra_mla_kv_assemble_bwd_vec_kernel(const uint4* __restrict__ dk, const uint4* __restrict__ dv,
                                     const int32_t* __restrict__ positions, uint4* __restrict__ dkv_up,
                                     uint4* __restrict__ dk_pe, int64_t n_tokens, int32_t n_heads, int32_t nope,
                                     int32_t rope_dim, int32_t dvd, double log_theta)
{
    __shared__ __align__(16) float s_cos[kMaxRopePairs], s_sin[kMaxRopePairs];
    const int nv = nope / 8, rv = rope_dim / 8, vv = dvd / 8;
    const int up_vecs = nv + vv, k_vecs = nv + rv;
    const double freq = exp(-log_theta * (2.0 * threadIdx.x) / rope_dim);
    for (int64_t t = blockIdx.x; t < n_tokens; t += gridDim.x) {
        __syncthreads();
        rope_table_fast(s_cos, s_sin, positions[t], rope_dim / 2, freq, 1);
        __syncthreads();
        const int64_t up0 = t * n_heads * up_vecs, k0 = t * n_heads * k_vecs, v0 = t * n_heads * vv;
        for (int e = threadIdx.x; e < n_heads * up_vecs; e += kRopeThreads) {
            const int a = e / up_vecs, c = e - a * up_vecs;
            dkv_up[up0 + e] = c < nv ? dk[k0 + static_cast<int64_t>(a) * k_vecs + c]
                                     : dv[v0 + static_cast<int64_t>(a) * vv + (c - nv)];
        }
        // the shared rotary key's gradient: the sum over the heads, in fp32, rotated back (one vector per thread)
        if (static_cast<int>(threadIdx.x) < rv) {
            const int i = threadIdx.x;
            float acc[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] = 0.f;
            for (int a = 0; a < n_heads; ++a) {
                const uint4 w = dk[k0 + static_cast<int64_t>(a) * k_vecs + nv + i];
                const uint32_t in[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float2 f = bf2_to_f2(in[j]);
                    acc[2 * j] += f.x;
                    acc[2 * j + 1] += f.y;
                }
            }
            uint32_t out[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float c = s_cos[4 * i + j], sn = s_sin[4 * i + j];
                out[j] = f2_to_bf2(acc[2 * j] * c - acc[2 * j + 1] * sn, acc[2 * j] * sn + acc[2 * j + 1] * c);
            }
            dk_pe[t * rv + i] = make_uint4(out[0], out[1], out[2], out[3]);
        }
    }
}

inline bool aligned16_all(std::initializer_list<const void*> ptrs)
{
    uintptr_t bits = 0;
    for (const void* p : ptrs) bits |= reinterpret_cast<uintptr_t>(p);
    return (bits & 15u) == 0;
}

// (exp and reciprocal of the special-function unit: a relative error of 2^-21, far below the bf16 result's 2^-9)
__device__ __forceinline__ float sigmoidf_(float x) { return __fdividef(1.f, 1.f + __expf(-x)); }

// kWords 32-bit words (pairs of bf16) per thread and access: 4 (16 bytes), or 8 (32 bytes) where the element
// count and the buffers allow it. Half as many threads then share the loop and address arithmetic.
template <int kWords>
struct Words { uint32_t w[kWords]; };
template <int kWords>
__device__ __forceinline__ Words<kWords> ld_words(const void* base, int64_t i)
{
    Words<kWords> v;
    if constexpr (kWords == 8) {
        const Words<8>* p = static_cast<const Words<8>*>(base) + i;
        asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]), "=r"(v.w[5]),
                       "=r"(v.w[6]), "=r"(v.w[7])
                     : "l"(p));
    } else {
        const uint4 t = static_cast<const uint4*>(base)[i];
        v.w[0] = t.x; v.w[1] = t.y; v.w[2] = t.z; v.w[3] = t.w;
    }
    return v;
}
template <int kWords>
__device__ __forceinline__ void st_words(void* base, int64_t i, const Words<kWords>& v)
{
    if constexpr (kWords == 8) {
        st_global_v8(static_cast<Words<8>*>(base) + i, v.w);
    } else {
        static_cast<uint4*>(base)[i] = make_uint4(v.w[0], v.w[1], v.w[2], v.w[3]);
    }
}

// y = out * sigmoid(gate)
template <int kWords>
__global__ void __launch_bounds__(256)
hydra_gate_kernel(const void* __restrict__ out, const void* __restrict__ gate, void* __restrict__ y, int64_t n)
{
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x; i < n; i += static_cast<int64_t>(gridDim.x) * 256) {
        const Words<kWords> o = ld_words<kWords>(out, i), g = ld_words<kWords>(gate, i);
        Words<kWords> r;
#pragma unroll
        for (int e = 0; e < kWords; ++e) {
            const float2 a = bf2_to_f2(o.w[e]), b = bf2_to_f2(g.w[e]);
            r.w[e] = f2_to_bf2(a.x * sigmoidf_(b.x), a.y * sigmoidf_(b.y));
        }
        st_words<kWords>(y, i, r);
    }
}

// d_out = dy * sigmoid(gate);  d_gate = dy * out * sigmoid(gate) * (1 - sigmoid(gate))
template <int kWords>
__global__ void __launch_bounds__(256)
hydra_gate_bwd_kernel(const void* __restrict__ dy, const void* __restrict__ out, const void* __restrict__ gate,
                      void* __restrict__ d_out, void* __restrict__ d_gate, int64_t n)
{
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x; i < n; i += static_cast<int64_t>(gridDim.x) * 256) {
        const Words<kWords> d = ld_words<kWords>(dy, i), o = ld_words<kWords>(out, i), g = ld_words<kWords>(gate, i);
        Words<kWords> ro, rg;
#pragma unroll
        for (int e = 0; e < kWords; ++e) {
            const float2 a = bf2_to_f2(d.w[e]), b = bf2_to_f2(o.w[e]), c = bf2_to_f2(g.w[e]);
            const float s0 = sigmoidf_(c.x), s1 = sigmoidf_(c.y);
            ro.w[e] = f2_to_bf2(a.x * s0, a.y * s1);
            rg.w[e] = f2_to_bf2(a.x * b.x * s0 * (1.f - s0), a.y * b.y * s1 * (1.f - s1));
        }
        st_words<kWords>(d_out, i, ro);
        st_words<kWords>(d_gate, i, rg);
    }
}

inline bool all_aligned32(std::initializer_list<const void*> ptrs)
{
    uintptr_t bits = 0;
    for (const void* p : ptrs) bits |= reinterpret_cast<uintptr_t>(p);
    return (bits & 31u) == 0;
}

int grid_for(int64_t work_items, int per_block)
{
    const int64_t blocks = (work_items + per_block - 1) / per_block;
    return static_cast<int>(blocks < 1 ? 1 : (blocks < 148 * 16 ? blocks : 148 * 16));
}

}  // namespace

cudaError_t launch_rope(const void* x, const int32_t* positions, void* y, int64_t n_tokens, int32_t n_heads,
                        int32_t head_dim, int32_t rope_offset, int32_t rope_dim, float theta, int inverse,
                        cudaStream_t stream)
{
    if (n_tokens == 0) return cudaSuccess;
    if (head_dim % 8 == 0 && rope_offset % 8 == 0 && rope_dim % 8 == 0 && rope_dim / 2 <= kRopeThreads &&
        aligned16_all({x, y})) {
        hydra_rope_vec_kernel<<<grid_for(n_tokens, 1), kRopeThreads, 0, stream>>>(
            static_cast<const uint4*>(x), positions, static_cast<uint4*>(y), n_tokens, n_heads, head_dim, rope_offset,
            rope_dim, std::log(static_cast<double>(theta)), inverse, x == y ? 1 : 0);
        return cudaGetLastError();
    }
    hydra_rope_kernel<<<grid_for(n_tokens, 1), kRopeThreads, 0, stream>>>(
        static_cast<const uint32_t*>(x), positions, static_cast<uint32_t*>(y), n_tokens, n_heads, head_dim, rope_offset,
        rope_dim, std::log(static_cast<double>(theta)), inverse, x == y ? 1 : 0);
    return cudaGetLastError();
}

cudaError_t launch_mla_kv_assemble(const void* kv_up, const void* k_pe, const int32_t* positions, void* k, void* v,
                                   int64_t n_tokens, int32_t n_heads, int32_t nope, int32_t rope_dim, int32_t dv,
                                   float theta, cudaStream_t stream)
{
    if (n_tokens == 0) return cudaSuccess;
    if (nope % 8 == 0 && rope_dim % 8 == 0 && dv % 8 == 0 && rope_dim / 2 <= kRopeThreads &&
        aligned16_all({kv_up, k_pe, k, v})) {
        hydra_mla_kv_assemble_vec_kernel<<<grid_for(n_tokens, 1), kRopeThreads, 0, stream>>>(
            static_cast<const uint4*>(kv_up), static_cast<const uint4*>(k_pe), positions, static_cast<uint4*>(k),
            static_cast<uint4*>(v), n_tokens, n_heads, nope, rope_dim, dv, std::log(static_cast<double>(theta)));
        return cudaGetLastError();
    }
    hydra_mla_kv_assemble_kernel<<<grid_for(n_tokens, 1), kRopeThreads, 0, stream>>>(
        static_cast<const uint32_t*>(kv_up), static_cast<const uint32_t*>(k_pe), positions, static_cast<uint32_t*>(k),
        static_cast<uint32_t*>(v), n_tokens, n_heads, nope, rope_dim, dv, std::log(static_cast<double>(theta)));
    return cudaGetLastError();
}

cudaError_t launch_mla_kv_assemble_bwd(const void* dk, const void* dv, const int32_t* positions, void* dkv_up,
                                       void* dk_pe, int64_t n_tokens, int32_t n_heads, int32_t nope, int32_t rope_dim,
                                       int32_t dvd, float theta, cudaStream_t stream)
{
    if (n_tokens == 0) return cudaSuccess;
    if (nope % 8 == 0 && rope_dim % 8 == 0 && dvd % 8 == 0 && rope_dim / 2 <= kRopeThreads &&
        aligned16_all({dk, dv, dkv_up, dk_pe})) {
        hydra_mla_kv_assemble_bwd_vec_kernel<<<grid_for(n_tokens, 1), kRopeThreads, 0, stream>>>(
            static_cast<const uint4*>(dk), static_cast<const uint4*>(dv), positions, static_cast<uint4*>(dkv_up),
            static_cast<uint4*>(dk_pe), n_tokens, n_heads, nope, rope_dim, dvd, std::log(static_cast<double>(theta)));
        return cudaGetLastError();
    }
    hydra_mla_kv_assemble_bwd_kernel<<<grid_for(n_tokens, 1), kRopeThreads, 0, stream>>>(
        static_cast<const uint32_t*>(dk), static_cast<const uint32_t*>(dv), positions, static_cast<uint32_t*>(dkv_up),
        static_cast<uint32_t*>(dk_pe), n_tokens, n_heads, nope, rope_dim, dvd, std::log(static_cast<double>(theta)));
    return cudaGetLastError();
}

cudaError_t launch_gate(const void* out, const void* gate, void* y, int64_t n8, cudaStream_t stream)
{
    if (n8 == 0) return cudaSuccess;
    if ((n8 & 1) == 0 && all_aligned32({out, gate, y}))
        hydra_gate_kernel<8><<<grid_for(n8 / 2, 256), 256, 0, stream>>>(out, gate, y, n8 / 2);
    else
        hydra_gate_kernel<4><<<grid_for(n8, 256), 256, 0, stream>>>(out, gate, y, n8);
    return cudaGetLastError();
}

cudaError_t launch_gate_bwd(const void* dy, const void* out, const void* gate, void* d_out, void* d_gate, int64_t n8,
                            cudaStream_t stream)
{
    if (n8 == 0) return cudaSuccess;
    if ((n8 & 1) == 0 && all_aligned32({dy, out, gate, d_out, d_gate}))
        hydra_gate_bwd_kernel<8><<<grid_for(n8 / 2, 256), 256, 0, stream>>>(dy, out, gate, d_out, d_gate, n8 / 2);
    else
        hydra_gate_bwd_kernel<4><<<grid_for(n8, 256), 256, 0, stream>>>(dy, out, gate, d_out, d_gate, n8);
    return cudaGetLastError();
}

}  // namespace hydra
