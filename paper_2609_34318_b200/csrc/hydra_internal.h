// Internal declarations shared by the host API and the kernel translation units.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/hydra_attn.h"

namespace hydra {

constexpr int D_QK = HYDRA_D_QK;
constexpr int D_V = HYDRA_D_V;
constexpr int TILE = 128;       // rows of a q tile and of a kv tile
constexpr int SUB = 64;         // rows of a q sub-tile in the key-side backward kernel
constexpr int FWD_SHORT_KEYS = 64;   // keys per step of the short-sequence forward kernel

// One (q-chunk, kv-chunk) pair with absolute token offsets, as the kernels see it.
struct PairDev {
    int32_t q_tok0;    // token index of the pair's first q row
    int32_t q_len;
    int32_t k_tok0;    // token index of the pair's first kv row
    int32_t k_len;
    int32_t off;       // q_start - k_start: key j is visible to q row i iff j <= i + off (causal)
    int32_t out_row0;  // first output row: part_row (partial buffers) or q_tok0 (out / lse)
    int32_t to_part;   // 1: partial buffers, 0: out / lse
    int32_t ds_base;   // backward: first block of this pair in the dS hand-off buffer (per head)
};

// Geometry of the dS hand-off buffer of the backward. The key-side kernel writes dS^T of every
// (128-row kv tile jk, 64-row q sub-tile u) it visits as one block of 16 KB: 8 chunks (8 q rows each) of
// 128 kv rows x 16 bytes, which is the tensor core's operand layout without swizzle (so the writer's
// stores are contiguous per warp and the reader's copy is one untiled bulk copy); the
// query-side kernel reads the blocks (jk, 2i) and (jk, 2i + 1) of its q tile i. Per pair the blocks of
// kv tile jk start at ds_rowstart(jk) and cover the sub-tiles ds_first(jk) .. nu_even - 1, where
// ds_first is the first sub-tile the causal mask leaves visible, rounded down to an even number, so
// that the buffer holds the visible trapezoid only. Both kernels and the host evaluate these forms.
struct DsGeom { int32_t nu_even; int32_t fo; };
__host__ __device__ inline DsGeom ds_geom(int32_t q_len, int32_t off, int causal)
{
    DsGeom g;
    g.nu_even = ((q_len + SUB - 1) / SUB + 1) & ~1;
    // fo = floor(-off / 128): kv tile jk sees q tiles jk + fo and later
    g.fo = !causal ? -(1 << 24) : (off <= 0 ? (-off) / TILE : -((off + TILE - 1) / TILE));
    return g;
}
__host__ __device__ inline int32_t ds_first(const DsGeom& g, int32_t jk)
{
    const int32_t m = jk + g.fo;
    return m > 0 ? 2 * m : 0;
}
__host__ __device__ inline int64_t ds_rowstart(const DsGeom& g, int32_t jk)
{
    int64_t m = static_cast<int64_t>(jk) + g.fo;
    if (m < 0) m = 0;
    const int64_t m0 = g.fo > 0 ? g.fo : 0;
    return static_cast<int64_t>(jk) * g.nu_even - (m * (m - 1) - m0 * (m0 - 1));
}
constexpr uint32_t DS_BLOCK_BYTES = TILE * SUB * 2;   // 16 KB

// Forward work item: up to 512 q rows of one pair and head = tiles A and B of 256 rows (128 per CTA of the pair).
struct FwdItem {
    int32_t pair;
    int32_t head;
    int32_t q0;        // first q row of tile A, relative to the pair; tile B starts at q0 + 128
    int32_t n_a;       // kv tiles tile A visits (after causal clipping); 0: its rows see no key
    int32_t n_b;       // same for tile B; -1 when the item has no second tile (its rows belong to another item)
    int32_t pad[3];
};

// Work item of the short-sequence forward kernel: one 128-row q tile of one pair and head, self-contained
// (a slot of that kernel reads nothing else to start it).
struct alignas(16) FwdShortItem {
    int32_t q_tok0;    // token index of the tile's first q row
    int32_t k_tok0;    // token index of the pair's first kv row
    int32_t k_len;
    int32_t off;       // key j is visible to row r of the tile iff j <= r + off (causal)
    int32_t out_row0;  // output row of the tile's first q row (partial buffers or out / lse)
    uint16_t head;
    uint16_t n_kv;     // steps of FWD_SHORT_KEYS keys the tile visits; 0: its rows see no key
    uint8_t rows;      // q rows of the tile that exist (1..128)
    uint8_t to_part;   // 1: partial buffers, 0: out / lse
    uint16_t pad;
    int32_t pad2;
};
static_assert(sizeof(FwdShortItem) == 32, "two 16-byte loads per work item");

// Backward work item: one tile of one chunk and head, visiting every pair that shares the chunk.
struct GroupItem {
    int32_t list_off;  // first entry of the chunk's pair list
    int32_t list_len;
    int32_t head;
    int32_t r0;        // first row of the tile, relative to the chunk
};

// Merge: one q chunk with two or more partials.
struct MergeGroup {
    int32_t out_tok0;  // first token of the chunk in out / lse
    int32_t rows;
    int32_t list_off;  // first entry of the chunk's part_row list
    int32_t n_parts;
};
struct MergeItem {
    int32_t group;
    int32_t row0;      // first row of the block, relative to the chunk
};
constexpr int MERGE_ROWS = 8;   // rows of a merge block

struct StatusBlock {            // lives at the start of the workspace; zeroed before every call
    int32_t status;
    int32_t pad;
    int64_t detail;
    int32_t next_item[4];       // work-queue heads of the persistent kernels (forward, dK/dV, dQ, short forward)
    // SM clock seen from inside the tensor-core kernels: cycles and nanoseconds that passed in the
    // producer thread of CTA 0 between its first and its last instruction (same index as next_item)
    uint64_t probe_cycles[4];
    uint64_t probe_ns[4];
};
enum : int { QUEUE_FWD = 0, QUEUE_DKV = 1, QUEUE_DQ = 2, QUEUE_FWD_SHORT = 3 };

#ifdef __CUDACC__
// The clock the driver reports between kernels says little about a 1 ms kernel on a power-capped part;
// the ratio of the cycle counter to the nanosecond timer inside the kernel does.
struct ClockProbe {
    long long c0; uint64_t t0;
    __device__ __forceinline__ void start()
    {
        c0 = clock64();
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    }
    __device__ __forceinline__ void stop(StatusBlock* sb, int queue) const
    {
        uint64_t t1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        sb->probe_cycles[queue] = static_cast<uint64_t>(clock64() - c0);
        sb->probe_ns[queue] = t1 - t0;
    }
};
#endif

struct FwdParams {
    const PairDev* pairs;
    const FwdItem* items;
    int32_t n_items;
    const FwdShortItem* short_items;   // the pairs that go to the short-sequence kernel
    int32_t n_short;
    void* out; float* lse; void* o_part; float* lse_part;
    int64_t T; int64_t part_rows;
    int32_t h; int32_t causal;
    int32_t kv_group;           // query heads per KV head (1: every head has its own K, V)
    float scale_log2;           // softmax_scale * log2(e)
    StatusBlock* status;
    uint64_t wait_limit_ns;
    uint64_t debug_stall_ns;    // test hook (hydra_debug_stall): 0 in normal operation
};

struct BwdParams {
    const PairDev* pairs;
    const int32_t* lists;       // pair indices, grouped by chunk
    const GroupItem* items;
    int32_t n_items;
    const float* lse; const float* dsum;   // [h, T]
    void* dq; void* dk; void* dv;   // bf16 [T,h,d], written; or, with accumulate, fp32 [T,h,d], added to
    int64_t T;
    int32_t h; int32_t causal;
    int32_t kv_group;           // query heads per KV head; k, v, dk, dv have h / kv_group heads
    float scale; float scale_log2;
    int32_t accumulate;
    void* ds;                   // dS hand-off buffer, or null: the query-side kernel recomputes S and dP
    int64_t ds_head_blocks;     // blocks per head
    StatusBlock* status;
    uint64_t wait_limit_ns;
    uint64_t debug_stall_ns;    // test hook (hydra_debug_stall): 0 in normal operation
};

struct MergeParams {
    const MergeGroup* groups;
    const int32_t* lists;       // part_row of every partial, grouped by chunk
    const MergeItem* items;
    int32_t n_items;
    const void* o_part; const float* lse_part;
    void* out; float* lse;
    int64_t T; int64_t part_rows;
    int32_t h;
    int32_t accumulate;         // 1: the current (out, lse) rows are one more input of their merge
    int32_t max_parts;          // most partials any chunk has (chooses how many are requested together)
};

// The tensor-core kernels exist once per supported q / k head dimension (the kernel files are compiled
// twice): the unsuffixed set for d_qk = 192, the _d128 set for d_qk = 128; d_v = 128 in both.
#define HYDRA_DECLARE_KERNEL_SET(SUFFIX)                                                                              \
    size_t fwd_smem_bytes##SUFFIX();                                                                                  \
    int fwd_max_clusters##SUFFIX();                                                                                   \
    size_t bwd_dq_smem_bytes##SUFFIX();                                                                               \
    size_t bwd_dkv_smem_bytes##SUFFIX();                                                                              \
    size_t bwd_dq_ds_smem_bytes##SUFFIX();                                                                            \
    cudaError_t launch_fwd##SUFFIX(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,               \
                                   const FwdParams& p, int grid, cudaStream_t stream);                                \
    size_t fwd_short_smem_bytes##SUFFIX();                                                                            \
    cudaError_t launch_fwd_short##SUFFIX(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv_sub,     \
                                         const FwdParams& p, int grid, cudaStream_t stream);                          \
    cudaError_t launch_bwd_dq##SUFFIX(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,            \
                                      const CUtensorMap& mdo, const BwdParams& p, int grid, cudaStream_t stream);     \
    cudaError_t launch_bwd_dq_from_ds##SUFFIX(const CUtensorMap& mk, const BwdParams& p, int grid,                    \
                                              cudaStream_t stream);                                                   \
    cudaError_t launch_bwd_dkv##SUFFIX(const CUtensorMap& mq_sub, const CUtensorMap& mk, const CUtensorMap& mv,       \
                                       const CUtensorMap& mdo_sub, const BwdParams& p, int grid, cudaStream_t stream);
HYDRA_DECLARE_KERNEL_SET()
HYDRA_DECLARE_KERNEL_SET(_d128)
#undef HYDRA_DECLARE_KERNEL_SET
cudaError_t launch_merge(const MergeParams& p, cudaStream_t stream);
// launch_merge plus the library's launch counter and per-kernel timer (defined beside them, in api.cu)
cudaError_t launch_merge_counted(const MergeParams& p, cudaStream_t stream);
cudaError_t launch_grad_cast(const float* acc, void* grad, int64_t n, cudaStream_t stream);
cudaError_t launch_ulysses(bool pack, const void* src, void* dst, int64_t n_tokens, int32_t cp_u, int64_t chunk_units,
                           cudaStream_t stream);
// the elementwise steps of a gated MLA block around the attention kernel (mla_ops.cu)
cudaError_t launch_rope(const void* x, const int32_t* positions, void* y, int64_t n_tokens, int32_t n_heads,
                        int32_t head_dim, int32_t rope_offset, int32_t rope_dim, float theta, int inverse,
                        cudaStream_t stream);
cudaError_t launch_mla_kv_assemble(const void* kv_up, const void* k_pe, const int32_t* positions, void* k, void* v,
                                   int64_t n_tokens, int32_t n_heads, int32_t nope, int32_t rope_dim, int32_t dv,
                                   float theta, cudaStream_t stream);
cudaError_t launch_mla_kv_assemble_bwd(const void* dk, const void* dv, const int32_t* positions, void* dkv_up,
                                       void* dk_pe, int64_t n_tokens, int32_t n_heads, int32_t nope, int32_t rope_dim,
                                       int32_t dvd, float theta, cudaStream_t stream);
cudaError_t launch_gate(const void* out, const void* gate, void* y, int64_t n8, cudaStream_t stream);
cudaError_t launch_gate_bwd(const void* dy, const void* out, const void* gate, void* d_out, void* d_gate, int64_t n8,
                            cudaStream_t stream);
cudaError_t launch_bwd_prep(const void* dout, const void* out, float* dsum, int64_t T, int32_t h,
                            cudaStream_t stream);

}  // namespace hydra
