/*
 * hydra_attn.h - C ABI of the B200 (sm_100a) attention library.
 *
 * The library computes the per-GPU work that HyDra's context-parallel engine schedules: causal
 * softmax attention, forward and backward, over variable-length packed sequences with one K/V head
 * per query head (MLA with materialised K/V; d_qk = 192, d_v = 128), cut into the (q-chunk,
 * kv-chunk) pairs of an outer ring, each pair emitting a partial (O, LSE), plus the log-sum-exp
 * merge of the partials.
 *
 * Conventions that hold for every entry point
 *   - "device" pointers are CUDA device memory of the current device, 16-byte aligned, contiguous;
 *     "host" pointers are ordinary host memory, read during the call and free to reuse on return.
 *   - Tensors: q, k, dq, dk [T, h, 192] bf16; v, out, dout, dv, o_part [rows, h, 128] bf16;
 *     lse [h, T] fp32, lse_part [h, part_rows] fp32 (natural logarithm, softmax scale included).
 *     T = cu_seqlens[n_seqs]; sequence b owns tokens [cu_seqlens[b], cu_seqlens[b+1]).
 *   - Every call returns a status (HYDRA_OK = 0). Work is enqueued on `cuda_stream` (a
 *     cudaStream_t passed as void*; NULL = the legacy default stream); results are valid once the
 *     stream has been synchronised. No call synchronises the device except hydra_poll_status,
 *     hydra_shutdown and the first compute call on a device, which allocates the library's table
 *     arena (see hydra_set_plan_arena_bytes): a new (cu_seqlens, pairs, h) combination costs host
 *     work and an asynchronous copy on `cuda_stream`, no allocation and no wait.
 *   - The caller owns all tensors and the workspace; the library keeps no caller pointer.
 *   - A workspace carries the status word and the work-queue counters of the kernels of one call:
 *     each call clears them (on its stream) before it launches, so calls that may run at the same
 *     time need workspaces of their own; calls on one stream may share one.
 *   - Inputs must be finite: a tile that straddles the end of a sequence reads (and masks) the
 *     rows of its neighbour, and 0 * NaN is NaN.
 *   - Only compute capability 10.0 is supported; there is no fallback path.
 */
#ifndef HYDRA_ATTN_H
#define HYDRA_ATTN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif
#if defined(__GNUC__)
#pragma GCC visibility push(default)
#endif

#define HYDRA_D_QK 192
#define HYDRA_D_V 128

enum {
    HYDRA_OK = 0,
    HYDRA_ERR_INVALID_ARG = 1,         /* null/misaligned pointer, bad cu_seqlens, bad pair      */
    HYDRA_ERR_UNSUPPORTED = 2,         /* shape outside the compiled configuration               */
    HYDRA_ERR_WORKSPACE_TOO_SMALL = 3,
    HYDRA_ERR_CUDA = 4,                /* a CUDA runtime/driver call failed                      */
    HYDRA_ERR_DEVICE_TIMEOUT = 5,      /* a bounded device-side wait gave up                     */
    HYDRA_ERR_NOT_SM100 = 6            /* current device is not compute capability 10.x          */
};

enum { HYDRA_WS_FWD = 0, HYDRA_WS_MERGE = 1, HYDRA_WS_BWD = 2 };

/*
 * One (q-chunk, kv-chunk) pair of one sequence: the unit of work of a ring step (Section 5.2: the
 * outer ring circulates K/V blocks and pipelines them with attention).  Offsets are local to the
 * sequence. With causal != 0 a key at position k_start+j is visible to the query at position
 * q_start+i iff k_start+j <= q_start+i (absolute positions; not "bottom-right aligned").
 */
typedef struct hydra_pair_t {
    int32_t seq;       /* index into cu_seqlens                                                    */
    int32_t q_start;   /* q rows  [q_start, q_start + q_len) of the sequence                       */
    int32_t q_len;
    int32_t k_start;   /* kv rows [k_start, k_start + k_len) of the sequence                       */
    int32_t k_len;
    int32_t part_row;  /* first row of this pair's partial in o_part / lse_part;                   */
                       /* -1: the pair is alone in its group and writes out / lse directly         */
    int32_t group;     /* merge group (the q chunk): pairs with equal ids share q_start/q_len and  */
                       /* are merged; ids are non-decreasing along the array                       */
    int32_t flags;     /* must be 0                                                                */
} hydra_pair_t;

/*
 * Eq. (usp), Section 5.2: a context-parallel degree P over h heads is run as an inner Ulysses
 * group cp_u = min(P, h) inside an outer ring cp_r = P / cp_u. The kernel of one rank then sees
 * H / cp_u heads and sequences cut into 2 * cp_r zigzag chunks.
 * Returns HYDRA_ERR_INVALID_ARG if degree or heads < 1 or cp_u does not divide degree.
 */
int32_t hydra_usp_factor(int32_t degree, int32_t heads, int32_t* cp_u, int32_t* cp_r);

/*
 * Chunk cutting and causal pair enumeration (host only, integers).
 * Sequence b is cut into n_c = 2*cp_r[b] contiguous chunks with boundaries floor(c*L/n_c)
 * (cp_r[b] == 0: not cut, one chunk); ring rank r owns chunks r and n_c-1-r; every pair
 * (q chunk, kv chunk) with kv chunk <= q chunk and both non-empty is emitted, q chunks in order.
 * Groups with one pair get part_row = -1, the others consecutive rows of the partial buffers.
 *   cu_seqlens_host [n_seqs+1] host; cp_r_host [n_seqs] host, or NULL to use cp_r_all everywhere.
 *   pairs_out       host array of capacity max_pairs (may be NULL with max_pairs = 0 to count).
 *   n_pairs_out     number of pairs (always written); part_rows_out rows needed in o_part/lse_part.
 *   rank_out, step_out  optional host arrays [max_pairs]: owner rank of the q chunk and ring step
 *                   (rank(q chunk) - rank(kv chunk)) mod cp_r at which the K/V block visits.
 * Returns HYDRA_ERR_INVALID_ARG on bad input, HYDRA_ERR_WORKSPACE_TOO_SMALL if max_pairs is too
 * small (counts are still written).
 */
int32_t hydra_zigzag_pairs(const int32_t* cu_seqlens_host, int32_t n_seqs, const int32_t* cp_r_host,
                           int32_t cp_r_all, hydra_pair_t* pairs_out, int32_t max_pairs,
                           int32_t* n_pairs_out, int64_t* part_rows_out, int32_t* rank_out,
                           int32_t* step_out);

/*
 * Bytes of device workspace the call `which` (HYDRA_WS_*) needs for this problem. pairs == NULL
 * with n_pairs == 0 means one whole-sequence pair per sequence. Returns 0 on invalid input.
 *
 * HYDRA_WS_BWD has two sizes. The backward always needs the status block and D (4 bytes per token
 * and head). If, in addition, the workspace has room for dS of every visible (query, key) position
 * as bf16 (2 bytes per position and head, laid out in 16 KB blocks), the key-side kernel hands dS to
 * the query-side kernel through the workspace and the latter computes dq = scale * dS k without
 * recomputing the scores (the backward then executes 1664 instead of 2304 FLOP per position). This
 * function returns the larger size while the hand-off buffer stays within the limit set with
 * hydra_set_bwd_scratch_limit (default 4 GiB; 0 switches the hand-off off) and the smaller size
 * otherwise; hydra_attn_bwd uses the hand-off whenever the workspace it is given is large enough and
 * the buffer is within the limit. The results of the two forms agree to the rounding of dS to bf16,
 * which both apply. The size assumes a causal call; a non-causal call needs about twice the buffer
 * and falls back to recomputation in a workspace sized here.
 *
 * Banded form, for problems whose dS buffer is over that limit (long sequences). The band scratch is set
 * with hydra_set_bwd_band_scratch(bytes): a byte count >= 1 MiB, 0 (bands off), or HYDRA_BAND_AUTO (the
 * default): as much as the dS limit, for problems whose whole dS buffer is at most 16 times the limit,
 * and off for larger ones (hundreds of small bands cost more than the recomputation they save: give
 * those an explicit scratch of tens of GB). With a scratch in effect HYDRA_WS_BWD asks, for a problem over
 * the limit, for the base size + an fp32 accumulator of dq (4 * 192 bytes per token and head) +
 * min(scratch, the full dS buffer). hydra_attn_bwd, given that much, cuts the key rows of every chunk into
 * bands of 128-row tiles whose own dS buffer fits the scratch and runs every band with the hand-off
 * (pairs clipped to the band's keys and, under the causal mask, to the query rows that see them). A key
 * tile lies in one band, so dk and dv come out as in the one-shot form; dq sums the bands' contributions
 * in fp32, band after band, and is rounded to bf16 once at the end. A problem that cannot be
 * banded (a single tile column over the scratch, or clipped chunks that would overlap without being
 * identical) runs in the recomputing form instead.
 */
#define HYDRA_BAND_AUTO (~(uint64_t)0)
void hydra_set_bwd_scratch_limit(uint64_t bytes);
void hydra_set_bwd_band_scratch(uint64_t bytes);

/*
 * Host only: the bands the banded backward would run for this problem with `scratch_bytes` of dS scratch.
 * Writes the clipped pairs of all bands, band after band, to pairs_out (capacity max_pairs; may be NULL
 * with max_pairs = 0 to count) and the band of each to band_out. Every visible (query, key) position of
 * the input pairs lies in exactly one clipped pair. n_bands_out = 0 means the problem cannot be banded
 * with that scratch. Returns HYDRA_ERR_WORKSPACE_TOO_SMALL if max_pairs is too small (counts are still
 * written), HYDRA_ERR_INVALID_ARG on bad input.
 */
int32_t hydra_bwd_bands(const int32_t* cu_seqlens_host, int32_t n_seqs, int32_t n_heads,
                        const hydra_pair_t* pairs, int32_t n_pairs, int32_t causal, uint64_t scratch_bytes,
                        hydra_pair_t* pairs_out, int32_t* band_out, int32_t max_pairs, int32_t* n_pairs_out,
                        int32_t* n_bands_out);
size_t hydra_workspace_bytes(int32_t which, const int32_t* cu_seqlens_host, int32_t n_seqs,
                             int32_t n_heads, const hydra_pair_t* pairs, int32_t n_pairs);

/*
 * Forward attention of every listed pair (the attention kernel of Section 3.5, restricted to one
 * ring step's blocks as in Section 5.2).  For pair p, head a and q row i:
 *   s_j = softmax_scale * <q_i, k_j> over the visible keys j of the pair,
 *   LSE = ln sum_j exp(s_j),  O = sum_j exp(s_j - LSE) v_j   (no visible key: O = 0, LSE = -inf).
 * Pairs with part_row >= 0 write rows [part_row, part_row+q_len) of o_part / lse_part, pairs with
 * part_row == -1 write their rows of out / lse.
 *   q, k, v device bf16; cu_seqlens_host, pairs host; out, lse, o_part, lse_part device (the
 *   partial buffers may be NULL when no pair uses them; out/lse likewise). part_rows = rows of the
 *   partial buffers. workspace device, >= hydra_workspace_bytes(HYDRA_WS_FWD, ...).
 * bf16 operands, fp32 accumulation. Rows not covered by any pair are left untouched.
 */
int32_t hydra_attn_fwd(const void* q, const void* k, const void* v, const int32_t* cu_seqlens_host,
                       int32_t n_seqs, int32_t n_heads, const hydra_pair_t* pairs, int32_t n_pairs,
                       int32_t causal, float softmax_scale, void* out, float* lse, void* o_part,
                       float* lse_part, int64_t part_rows, void* workspace, size_t workspace_bytes,
                       void* cuda_stream);

/*
 * Log-sum-exp merge of the partials of every group whose pairs carry partial rows (the combination step
 * of ring attention, Section 5.2):  LSE = ln sum_p exp(LSE_p),  O = sum_p exp(LSE_p - LSE) O_p,
 * all n partials at once in fp32 with one rounding to bf16; a partial with LSE_p = -inf has weight
 * zero; all -inf gives O = 0, LSE = -inf. Writes the group's rows of out / lse.
 *   o_part, lse_part device (as written by hydra_attn_fwd); out, lse device.
 */
int32_t hydra_lse_merge(const void* o_part, const float* lse_part, int64_t part_rows,
                        const int32_t* cu_seqlens_host, int32_t n_seqs, int32_t n_heads,
                        const hydra_pair_t* pairs, int32_t n_pairs, void* out, float* lse,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The same merge in its streaming form, one ring step at a time (Section 5.2, outer ring): after
 * every ring step the partials of that step are folded into the running (out, lse) of their q chunks,
 *   (out, lse) <- (out, lse) (+) partial_1 (+) ... (+) partial_n,
 * where (+) is the two-way form of the merge above; rows of out / lse that belong to no listed
 * group are left untouched. The first step of a chunk uses hydra_lse_merge (which accepts groups
 * of a single partial) or starts from out = 0, lse = -inf. The running out is stored as bf16, so
 * every step rounds it once; the result equals the one-shot merge up to those roundings.
 * Arguments as for hydra_lse_merge; out and lse are read and written.
 */
int32_t hydra_lse_merge_accumulate(const void* o_part, const float* lse_part, int64_t part_rows,
                                   const int32_t* cu_seqlens_host, int32_t n_seqs, int32_t n_heads,
                                   const hydra_pair_t* pairs, int32_t n_pairs, void* out, float* lse,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * hydra_lse_merge for callers that must not allocate device memory. (No counterpart in the paper:
 * this is a property of the library, not of the method.) It computes exactly what hydra_lse_merge
 * computes, with the same kernel, but keeps the per-problem tables (the partials of every q chunk,
 * cut into blocks of rows) in a fixed array inside the library image instead of in the arena that the
 * other entry points obtain with cudaMalloc at their first call, and it needs no workspace. It calls no cudaMalloc, cudaFree or other allocating
 * routine. It is meant for processes that have handed all device memory to their own pool, and for
 * latency-critical loops whose rules forbid cudaMalloc because it may synchronise the device.
 *   - Limits (HYDRA_ERR_UNSUPPORTED beyond them): at most HYDRA_NOALLOC_MAX_GROUPS merged q chunks,
 *     HYDRA_NOALLOC_MAX_PARTIALS partials in total, and HYDRA_NOALLOC_MAX_BLOCKS blocks of 8 rows
 *     (sum over merged chunks of ceil(q_len / 8)). The array takes 608 KB on every GPU that loads
 *     the library, until the process exits.
 *   - The first call on a device looks up the array's device address with that device current; make
 *     that first call before any stream capture begins.
 *   - No call may be made while `cuda_stream` is capturing: the tables travel from static host arrays
 *     that the next call overwrites, which a captured copy would read again at every replay. Such a
 *     call is refused with HYDRA_ERR_UNSUPPORTED before anything is touched.
 *   - All calls on a device share the one array and each call rewrites the part it uses: calls
 *     enqueued on the same stream are safe, calls whose kernels may overlap on the GPU (different
 *     streams, no dependency) race. The tables are copied from ordinary host memory, so the call
 *     waits for earlier work on `cuda_stream` before it returns; the host-side tables are one set
 *     per process behind one lock, so calls from several threads (also for different GPUs) take
 *     turns, each holding the lock through that wait.
 *   - As hydra_lse_merge, it refuses (HYDRA_ERR_INVALID_ARG) partial rows that overlap and merged q
 *     chunks whose output rows overlap.
 *   Arguments as for hydra_lse_merge (pairs with part_row == -1 are ignored).
 */
#define HYDRA_NOALLOC_MAX_GROUPS 2048
#define HYDRA_NOALLOC_MAX_PARTIALS 16384
#define HYDRA_NOALLOC_MAX_BLOCKS 65536
int32_t hydra_lse_merge_noalloc(const void* o_part, const float* lse_part, int64_t part_rows,
                                const int32_t* cu_seqlens_host, int32_t n_seqs, int32_t n_heads,
                                const hydra_pair_t* pairs, int32_t n_pairs, void* out, float* lse,
                                void* cuda_stream);

/*
 * Backward of the listed pairs, given the MERGED out and lse and the upstream gradient dout:
 *   D_i = <dout_i, out_i>;  P_ij = exp(s_ij - LSE_i);  dS_ij = P_ij (<dout_i, v_j> - D_i);
 *   dq_i = scale sum_j dS_ij k_j;  dk_j = scale sum_i dS_ij q_i;  dv_j = sum_i P_ij dout_i,
 * summed over all listed pairs that contain (i, j). The sums are accumulated on chip in fp32 and
 * written once as bf16, so results are deterministic. Rows of dq covered by no q chunk and rows of
 * dk/dv covered by no kv chunk are left untouched.
 * Requirement: any two pairs of a sequence have q ranges that are identical or disjoint, and kv
 * ranges that are identical or disjoint (true for chunk pairs); otherwise HYDRA_ERR_INVALID_ARG.
 *   q, k, v, out, dout device bf16; lse device fp32; dq, dk, dv device bf16.
 */
int32_t hydra_attn_bwd(const void* q, const void* k, const void* v, const void* out,
                       const float* lse, const void* dout, const int32_t* cu_seqlens_host,
                       int32_t n_seqs, int32_t n_heads, const hydra_pair_t* pairs, int32_t n_pairs,
                       int32_t causal, float softmax_scale, void* dq, void* dk, void* dv,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The backward of one ring step (Section 5.2, outer ring: a rank meets its chunk pairs a step at a
 * time, as the visiting K/V chunks arrive): the same computation as hydra_attn_bwd for the listed pairs, but the contributions are ADDED to fp32
 * accumulators instead of being written as bf16, so that calls for the successive steps sum to the
 * backward of all pairs. The paper does not print this form; it is what its ring engine needs from
 * the attention library.
 *   dq_acc, dk_acc  device fp32 [T, h, 192]; dv_acc device fp32 [T, h, 128]; the caller zeroes them
 *                   (or loads them with gradients that arrived from a peer) before the first step.
 *   out, lse        the MERGED forward result of all steps, as for hydra_attn_bwd.
 * Rows covered by no listed chunk are left untouched. The additions are fp32 reductions performed at
 * the L2 cache (red.global.add). Each accumulator address receives exactly one addition per call
 * (one thread block owns the row) and calls on one stream are ordered, so the result of a fixed
 * sequence of per-head calls does not depend on timing. (The grouped-query form is the exception:
 * the query heads of a group add into the same dk / dv rows in no fixed order.) Calls that share accumulators must be enqueued on one
 * stream (or ordered by the caller). Workspace, requirements and errors as for hydra_attn_bwd.
 * hydra_grad_cast converts an accumulator to the bf16 gradient: grad[i] = bf16(acc[i]), i <
 * n_elements (round to nearest even); acc, grad device pointers, 16-byte aligned.
 */
int32_t hydra_attn_bwd_accumulate(const void* q, const void* k, const void* v, const void* out,
                                  const float* lse, const void* dout, const int32_t* cu_seqlens_host,
                                  int32_t n_seqs, int32_t n_heads, const hydra_pair_t* pairs,
                                  int32_t n_pairs, int32_t causal, float softmax_scale, float* dq_acc,
                                  float* dk_acc, float* dv_acc, void* workspace, size_t workspace_bytes,
                                  void* cuda_stream);
int32_t hydra_grad_cast(const float* acc, void* grad, int64_t n_elements, void* cuda_stream);

/*
 * Grouped-query form (Table "Notation": h query heads and h_kv KV heads per rank; the GQA model of
 * Section 6 shares eight KV heads). With g = n_heads / n_kv_heads, query head a reads KV head a / g
 * (integer division); n_kv_heads must divide n_heads. k device bf16 [T, n_kv_heads, 192], v device bf16
 * [T, n_kv_heads, 128]; everything else as in hydra_attn_fwd / hydra_attn_bwd_accumulate, which are the
 * case n_kv_heads == n_heads.
 * In the backward dk, dv of a KV head are the SUM over the g query heads that read it: the work items of
 * the g query heads add into the same fp32 rows with reductions, so the order of the g terms, and with it
 * the last bits of dk / dv, may differ from run to run.
 *   hydra_attn_bwd_accumulate_gqa  dq_acc device fp32 [T, n_heads, 192], dk_acc device fp32
 *                                  [T, n_kv_heads, 192], dv_acc device fp32 [T, n_kv_heads, 128]: the
 *                                  caller zeroes them and rounds them with hydra_grad_cast.
 *   hydra_attn_bwd_gqa             one shot: dq device bf16 [T, n_heads, 192], dk device bf16
 *                                  [T, n_kv_heads, 192], dv device bf16 [T, n_kv_heads, 128]. dk and dv are
 *                                  summed in fp32 in the workspace and rounded once; the workspace must
 *                                  have hydra_workspace_bytes_gqa(HYDRA_WS_BWD, ...) bytes (the per-head
 *                                  size plus 4 * (192 + 128) bytes per token and KV head), else
 *                                  HYDRA_ERR_WORKSPACE_TOO_SMALL. The banded form does not apply.
 */
size_t hydra_workspace_bytes_gqa(int32_t which, const int32_t* cu_seqlens_host, int32_t n_seqs, int32_t n_heads,
                                 int32_t n_kv_heads, const hydra_pair_t* pairs, int32_t n_pairs);
int32_t hydra_attn_bwd_gqa(const void* q, const void* k, const void* v, const void* out, const float* lse,
                           const void* dout, const int32_t* cu_seqlens_host, int32_t n_seqs, int32_t n_heads,
                           int32_t n_kv_heads, const hydra_pair_t* pairs, int32_t n_pairs, int32_t causal,
                           float softmax_scale, void* dq, void* dk, void* dv, void* workspace,
                           size_t workspace_bytes, void* cuda_stream);
int32_t hydra_attn_fwd_gqa(const void* q, const void* k, const void* v, const int32_t* cu_seqlens_host,
                           int32_t n_seqs, int32_t n_heads, int32_t n_kv_heads, const hydra_pair_t* pairs,
                           int32_t n_pairs, int32_t causal, float softmax_scale, void* out, float* lse,
                           void* o_part, float* lse_part, int64_t part_rows, void* workspace,
                           size_t workspace_bytes, void* cuda_stream);
int32_t hydra_attn_bwd_accumulate_gqa(const void* q, const void* k, const void* v, const void* out,
                                      const float* lse, const void* dout, const int32_t* cu_seqlens_host,
                                      int32_t n_seqs, int32_t n_heads, int32_t n_kv_heads,
                                      const hydra_pair_t* pairs, int32_t n_pairs, int32_t causal,
                                      float softmax_scale, float* dq_acc, float* dk_acc, float* dv_acc,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The whole step (forward of every pair, merge, backward; Sections 3.5 and 5.2 as above) with HOST
 * buffers: copies q, k, v, dout to the device, runs hydra_attn_fwd, hydra_lse_merge (if any pair has
 * partial rows) and hydra_attn_bwd, and copies out, lse, dq, dk, dv back. Sequences and heads are
 * independent, so the step is pipelined over groups: runs of whole sequences with all heads
 * (contiguous on the host) when every sequence is small against the step, else groups of 2 or 4
 * heads over all sequences (with 4 or more heads). The kernels run on
 * `cuda_stream`, the copies in and out on two internal streams (created once per device, on the
 * first call), so that both directions of the host link are busy at once. Work enqueued on
 * `cuda_stream` before the call precedes all of it, and `cuda_stream` completes only when the last
 * copy out has: host outputs are valid once the stream has been synchronised. Host buffers have
 * the tensor layouts above; pinned memory makes the copies asynchronous. `device_arena` is device
 * memory, 256-byte aligned, of at least hydra_host_step_arena_bytes(...) bytes, owned by the
 * caller; the library carves every device tensor, the partial buffers and the workspace out of it
 * and allocates no device memory itself. One call at a time per device (the internal streams and
 * events are shared).
 */
size_t hydra_host_step_arena_bytes(const int32_t* cu_seqlens_host, int32_t n_seqs, int32_t n_heads,
                                   const hydra_pair_t* pairs, int32_t n_pairs);
int32_t hydra_attn_fwd_bwd_host(const void* q_host, const void* k_host, const void* v_host,
                                const void* dout_host, const int32_t* cu_seqlens_host, int32_t n_seqs,
                                int32_t n_heads, const hydra_pair_t* pairs, int32_t n_pairs,
                                int32_t causal, float softmax_scale, void* out_host, float* lse_host,
                                void* dq_host, void* dk_host, void* dv_host, void* device_arena,
                                size_t arena_bytes, void* cuda_stream);

/*
 * The same entry points with the head dimensions as arguments. Two pairs are built: d_qk = 192, d_v = 128
 * (the multi-head-latent model the configurations name: every other entry point is this case) and
 * d_qk = d_v = 128 (the grouped-query model of the scale-out simulation, Section 6: eight KV heads; the
 * paper gives no head dimension for it, 128 is the customary one). Any other pair returns
 * HYDRA_ERR_UNSUPPORTED (hydra_workspace_bytes_dims: 0). q, k and dq, dk then have d_qk columns per head,
 * v, out, dout and dv have d_v; everything else (layouts, partial buffers, workspace rules, banded and
 * grouped-query forms, errors) is as in the entry points without the suffix.
 */
size_t hydra_workspace_bytes_dims(int32_t which, const int32_t* cu_seqlens_host, int32_t n_seqs, int32_t n_heads,
                                  int32_t n_kv_heads, int32_t d_qk, int32_t d_v, const hydra_pair_t* pairs,
                                  int32_t n_pairs);
int32_t hydra_attn_fwd_dims(const void* q, const void* k, const void* v, const int32_t* cu_seqlens_host,
                            int32_t n_seqs, int32_t n_heads, int32_t n_kv_heads, int32_t d_qk, int32_t d_v,
                            const hydra_pair_t* pairs, int32_t n_pairs, int32_t causal, float softmax_scale,
                            void* out, float* lse, void* o_part, float* lse_part, int64_t part_rows,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);
int32_t hydra_attn_bwd_dims(const void* q, const void* k, const void* v, const void* out, const float* lse,
                            const void* dout, const int32_t* cu_seqlens_host, int32_t n_seqs, int32_t n_heads,
                            int32_t n_kv_heads, int32_t d_qk, int32_t d_v, const hydra_pair_t* pairs,
                            int32_t n_pairs, int32_t causal, float softmax_scale, void* dq, void* dk, void* dv,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);
int32_t hydra_attn_bwd_accumulate_dims(const void* q, const void* k, const void* v, const void* out,
                                       const float* lse, const void* dout, const int32_t* cu_seqlens_host,
                                       int32_t n_seqs, int32_t n_heads, int32_t n_kv_heads, int32_t d_qk,
                                       int32_t d_v, const hydra_pair_t* pairs, int32_t n_pairs, int32_t causal,
                                       float softmax_scale, float* dq_acc, float* dk_acc, float* dv_acc,
                                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Local layouts: what a rank of an outer ring calls (Section 5.2: the outer ring circulates K/V chunks and
 * pipelines with attention; Section 3.5, Eq. (ring)). Such a rank holds only its own q chunks and, at a ring
 * step, the visiting kv chunks; its tensors are not the packed batch. A chunk table says where the chunks of
 * the sequences sit:
 *   hydra_chunk_t { seq, start, len, row }   positions [start, start + len) of sequence seq occupy rows
 *                                            [row, row + len) of the tensor
 * q_chunks describes the q-side tensors (q, out, lse, dout, dq: q_rows rows; lse is [n_heads, q_rows]),
 * kv_chunks the kv-side tensors (k, v, dk, dv: kv_rows rows). The pairs keep their sequence-local positions
 * (the causal mask needs them); every pair's q range must lie inside one q chunk and its kv range inside one
 * kv chunk, chunks of one table must not share rows (else HYDRA_ERR_INVALID_ARG). cu_seqlens_host still gives
 * the lengths of the whole sequences. Everything else is as in hydra_attn_fwd_dims / hydra_lse_merge(_accumulate)
 * / hydra_attn_bwd_accumulate_dims: the forward of a step's pairs writes partials (or out / lse directly for a
 * chunk with one pair), the merge folds them into the running (out, lse) when `accumulate` is non-zero, the
 * backward adds the step's contributions into fp32 accumulators laid out like the tensors they belong to
 * (dq_acc with q_rows rows; dk_acc, dv_acc with kv_rows rows: they travel round the ring with their chunks).
 * The exchange of the chunks between the GPUs is the caller's (a peer copy or NCCL send / receive into this
 * GPU's own memory before the call: the kernels only ever read local memory).
 */
typedef struct {
    int32_t seq;
    int32_t start, len;
    int32_t row;
} hydra_chunk_t;
size_t hydra_workspace_bytes_local(int32_t which, const int32_t* cu_seqlens_host, int32_t n_seqs, int32_t n_heads,
                                   int32_t n_kv_heads, int32_t d_qk, int32_t d_v, const hydra_chunk_t* q_chunks,
                                   int32_t n_q_chunks, int64_t q_rows, const hydra_chunk_t* kv_chunks,
                                   int32_t n_kv_chunks, int64_t kv_rows, const hydra_pair_t* pairs, int32_t n_pairs);
int32_t hydra_attn_fwd_local(const void* q, const void* k, const void* v, const int32_t* cu_seqlens_host,
                             int32_t n_seqs, int32_t n_heads, int32_t n_kv_heads, int32_t d_qk, int32_t d_v,
                             const hydra_chunk_t* q_chunks, int32_t n_q_chunks, int64_t q_rows,
                             const hydra_chunk_t* kv_chunks, int32_t n_kv_chunks, int64_t kv_rows,
                             const hydra_pair_t* pairs, int32_t n_pairs, int32_t causal, float softmax_scale,
                             void* out, float* lse, void* o_part, float* lse_part, int64_t part_rows,
                             void* workspace, size_t workspace_bytes, void* cuda_stream);
int32_t hydra_lse_merge_local(const void* o_part, const float* lse_part, int64_t part_rows,
                              const int32_t* cu_seqlens_host, int32_t n_seqs, int32_t n_heads,
                              const hydra_chunk_t* q_chunks, int32_t n_q_chunks, int64_t q_rows,
                              const hydra_pair_t* pairs, int32_t n_pairs, int32_t accumulate, void* out, float* lse,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);
int32_t hydra_attn_bwd_accumulate_local(const void* q, const void* k, const void* v, const void* out,
                                        const float* lse, const void* dout, const int32_t* cu_seqlens_host,
                                        int32_t n_seqs, int32_t n_heads, int32_t n_kv_heads, int32_t d_qk,
                                        int32_t d_v, const hydra_chunk_t* q_chunks, int32_t n_q_chunks,
                                        int64_t q_rows, const hydra_chunk_t* kv_chunks, int32_t n_kv_chunks,
                                        int64_t kv_rows, const hydra_pair_t* pairs, int32_t n_pairs, int32_t causal,
                                        float softmax_scale, float* dq_acc, float* dk_acc, float* dv_acc,
                                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The local halves of the Ulysses all-to-all (Section 3.5: all-to-all transposes partition the attention
 * heads across the cp_u ranks of a group; Eq. (ulysses) counts the volume, about 4 S h / P elements per
 * rank for q, k, v and the output). Elements are 2 bytes wide (bf16) and are moved, not interpreted.
 *   hydra_ulysses_pack    x device [n_tokens, n_heads, head_dim] (this rank's tokens, all heads)
 *                         -> send device [cp_u, n_tokens, n_heads / cp_u, head_dim]:
 *                         send[j, t, b, :] = x[t, j * (n_heads / cp_u) + b, :]; block j goes to rank j.
 *                         With equal n_tokens on every rank the received buffer is
 *                         [cp_u * n_tokens, n_heads / cp_u, head_dim], tokens in rank order: the layout
 *                         hydra_attn_fwd takes, without another copy.
 *   hydra_ulysses_unpack  recv device [cp_u, n_tokens, n_heads / cp_u, head_dim] (block j from rank j: this
 *                         rank's tokens, rank j's heads) -> y device [n_tokens, n_heads, head_dim], the
 *                         inverse permutation (the way back after attention; on that way the split by
 *                         token owner before the exchange is contiguous and needs no kernel).
 * Requirements: cp_u divides n_heads; (n_heads / cp_u) * head_dim * 2 is a multiple of 16 bytes (else
 * HYDRA_ERR_UNSUPPORTED, as is a tensor of more than 60 GB); pointers 16-byte aligned, distinct buffers (not
 * in place). One kernel launch on
 * cuda_stream, HBM-bound: 4 bytes moved per element. HYDRA_ERR_INVALID_ARG on bad arguments.
 */
int32_t hydra_ulysses_pack(const void* x, int64_t n_tokens, int32_t n_heads, int32_t head_dim, int32_t cp_u,
                           void* send, void* cuda_stream);
int32_t hydra_ulysses_unpack(const void* recv, int64_t n_tokens, int32_t n_heads, int32_t head_dim, int32_t cp_u,
                             void* y, void* cuda_stream);

/*
 * The elementwise steps of a gated multi-head-latent attention block that surround the attention kernel
 * (Section 5.2, "Exposed All-to-All Overlap": the query's rotary embedding; the KV up-projection's output
 * split into the value and the key's position-free part; the key's rotary embedding and concatenation; the
 * gate). The paper names the steps and the order in which their results become final, not their formulas;
 * the readings taken here:
 *   rotary embedding  the columns [rope_offset, rope_offset + rope_dim) of every head are rotated in pairs
 *                     (2i, 2i+1) by the angle positions[t] * theta^(-2i / rope_dim):
 *                       y_2i = x_2i cos - x_2i+1 sin,  y_2i+1 = x_2i sin + x_2i+1 cos;
 *                     positions[t] is the token's index inside its packed sequence; inverse != 0 rotates by
 *                     the opposite angle, which is the backward of the step (a rotation's adjoint).
 *   key / value       the up-projection emits, per token and head, [d_nope key columns | d_v value columns];
 *                     the rotary part of the key is ONE vector of d_rope columns per token, shared by all
 *                     heads: k[t, a, :] = [kv_up[t, a, 0:d_nope] | rope(k_pe[t, :])], v[t, a, :] =
 *                     kv_up[t, a, d_nope:]. With d_nope = 128, d_rope = 64, d_v = 128 these are the
 *                     [T, h, 192] / [T, h, 128] tensors hydra_attn_fwd takes. The backward is the adjoint:
 *                     dkv_up = [dk[.., 0:d_nope] | dv], dk_pe[t, :] = rope^-1(sum_a dk[t, a, d_nope:]) (the sum
 *                     over the heads in fp32, rounded once).
 *   gate              y = out * sigmoid(gate), elementwise, gate being the gate projection's output with the
 *                     shape of out; backward d_out = dy * sigmoid(gate), d_gate = dy * out * sigmoid(gate) *
 *                     (1 - sigmoid(gate)).
 * All tensors device bf16, positions device int32 [n_tokens]; arithmetic in fp32 (the rotary angle is formed
 * and reduced in double precision), one rounding per output element. hydra_mla_rope may run in place (y == x);
 * all other outputs must not alias inputs. Dimensions must be even, rope_dim <= 256, theta > 1; the gate
 * takes n_elements % 8 == 0 and 16-byte aligned pointers (else HYDRA_ERR_INVALID_ARG). One launch each on
 * cuda_stream, bound by HBM: every byte moves once.
 */
int32_t hydra_mla_rope(const void* x, const int32_t* positions, int64_t n_tokens, int32_t n_heads, int32_t head_dim,
                       int32_t rope_offset, int32_t rope_dim, float theta, int32_t inverse, void* y,
                       void* cuda_stream);
int32_t hydra_mla_kv_assemble(const void* kv_up, const void* k_pe, const int32_t* positions, int64_t n_tokens,
                              int32_t n_heads, int32_t d_nope, int32_t d_rope, int32_t d_v, float theta, void* k,
                              void* v, void* cuda_stream);
int32_t hydra_mla_kv_assemble_bwd(const void* dk, const void* dv, const int32_t* positions, int64_t n_tokens,
                                  int32_t n_heads, int32_t d_nope, int32_t d_rope, int32_t d_v, float theta,
                                  void* dkv_up, void* dk_pe, void* cuda_stream);
int32_t hydra_gate_apply(const void* out, const void* gate, int64_t n_elements, void* y, void* cuda_stream);
int32_t hydra_gate_apply_bwd(const void* dy, const void* out, const void* gate, int64_t n_elements, void* d_out,
                             void* d_gate, void* cuda_stream);

/*
 * Per-kernel timing (measurement aid, not part of the method). While enabled, every kernel launch
 * is bracketed by CUDA events on its stream. hydra_profile_collect waits for the recorded events,
 * adds their durations into ms_out[8] and their counts into launches_out[8] (index: 0 forward, both of its
 * kernels when a call uses both,
 * 1 merge, 2 backward prep, 3 backward dK/dV, 4 backward dQ, 5 gradient cast, 6 Ulysses pack / unpack,
 * 7 the elementwise steps of the gated MLA block)
 * and forgets them.
 */
void hydra_profile_enable(int32_t on);
int32_t hydra_profile_collect(double* ms_out, int64_t* launches_out);

/* Human-readable name of a status code (static storage). */
const char* hydra_status_string(int32_t status);

/*
 * Synchronises `cuda_stream` and reports what the kernels of the last call that used `workspace`
 * left in its status word: *device_status is HYDRA_OK or HYDRA_ERR_DEVICE_TIMEOUT, *detail the
 * index of the work item that gave up (or -1). Returns HYDRA_ERR_CUDA if the stream is in error.
 * A workspace that no call has launched kernels with (none yet, or only calls without any token or pair, which
 * launch nothing) holds whatever the caller put there: zero it at allocation if it may be polled in that state.
 */
int32_t hydra_poll_status(void* workspace, void* cuda_stream, int32_t* device_status,
                          int64_t* detail);

/*
 * SM clock seen from inside the kernels of the last call that used `workspace` (measurement aid, not
 * part of the method). The producer thread of thread block 0 of every tensor-core kernel reads the
 * cycle counter and the nanosecond timer when it starts and when it has issued its last load;
 * mhz_out[3] receives cycles / microsecond for the forward, the key-side backward and the query-side
 * backward kernel (0 for a kernel the call did not run; the forward's figure is the CTA-pair kernel's if the
 * call used it, else the short-sequence kernel's). Synchronises the stream. On a power-capped
 * part this is the clock the kernel really ran at; the driver's clock query, sampled between
 * kernels, is not.
 */
int32_t hydra_poll_clocks(void* workspace, void* cuda_stream, double* mhz_out);

/* Kernel launches issued by this process so far (all entry points), for launch accounting. */
int64_t hydra_launch_count(void);

/*
 * Debug knob: upper bound, in nanoseconds, of any single device-side wait (default 2e9). Waits that
 * exceed it make the kernel record HYDRA_ERR_DEVICE_TIMEOUT and return.
 */
void hydra_set_wait_limit_ns(uint64_t ns);

/*
 * Test hook for the bounded waits above (no counterpart in the paper: it is how the library's own
 * failure path is exercised without faulting a GPU). While `ns` is non-zero for a
 * kernel, the thread of every thread block that hands out work items idles for `ns` nanoseconds
 * (at most 20 ms) at the start of that kernel's next launches and then hands out nothing and loads
 * nothing: the other roles wait for a signal that is never given, their waits run out at the limit set
 * with hydra_set_wait_limit_ns, the kernel records HYDRA_ERR_DEVICE_TIMEOUT with the index of a thread
 * block in `detail` and returns by itself (no trap, no endless loop, nothing in flight). Outputs of such
 * a launch are not written. ns = 0 (the default) switches the hook off; it costs one predicate per launch.
 */
#define HYDRA_STALL_FWD 0       /* either forward kernel */
#define HYDRA_STALL_BWD_DKV 1
#define HYDRA_STALL_BWD_DQ 2    /* either form of the query-side kernel */
void hydra_debug_stall(int32_t kernel, uint64_t ns);

int32_t hydra_version(void);

/*
 * Device memory the library itself owns. The work tables of a problem (pairs, work items, lists) are built
 * on the host, cached by content, and copied on the caller's stream (cudaMemcpyAsync from pinned staging)
 * into a table arena that is allocated ONCE per device, by the first compute call on that device (default
 * 32 MiB; hydra_set_plan_arena_bytes changes the size used by the next first call or the first call after
 * hydra_shutdown). After that first call no entry point allocates or frees device memory or waits for the
 * device, however many distinct problems are seen: when the arena is full its older half is recycled, and
 * the stream that recycles it waits on the device for the kernels that last read it. The one exception is a
 * problem whose tables exceed half the arena (about 500 000 work items at the default size): it gets an
 * allocation of its own, once. A first call on a device should precede any stream capture.
 * hydra_shutdown waits for the device and frees the arena, the cached tables and the pinned staging.
 */
void hydra_set_plan_arena_bytes(uint64_t bytes);
/*
 * In training the forward of a problem is followed by its merge and its backward. hydra_attn_fwd therefore
 * builds, on the host and right after it has launched its kernel, the work tables those calls will ask for
 * (if they are not cached yet), so that this host work runs while the GPU computes the forward. Nothing is
 * uploaded and no result changes. on = 0 switches it off (forward-only use); the default is on.
 */
void hydra_set_plan_prefetch(int32_t on);
/*
 * The forward has two kernels. Pairs whose q range AND kv range are at most `len` tokens long go to the
 * short-sequence kernel (one CTA per SM, two independent 128-row q tiles in flight, steps of 64 keys: the
 * regime of Section 2.2, where most sequences are short and a tile's chain of dependent steps, not the tensor
 * core, sets the pace), all others to the CTA-pair kernel; if the short pairs carry less than a quarter of a
 * call's work, that call uses the CTA-pair kernel alone. Both compute the same function to the same tolerance
 * (not bit for bit: their summation orders differ). len = 0 switches the short-sequence kernel off; a negative
 * len (the default) lets the library choose: 2048 for heads of 192 with a K / V head per query head, 4608 with
 * shared K / V heads or heads of 128 (where the kernels were measured to take equal time on sequences of one
 * length). Takes effect with the next call.
 */
void hydra_set_fwd_short_len(int32_t len);
/*
 * Host only (no GPU needed): seconds the host takes to build the work tables of one call of kind `which`
 * (HYDRA_WS_FWD / MERGE / BWD) for this problem, uncached. What a new cu_seqlens costs before its first launch.
 * Negative on invalid arguments.
 */
double hydra_plan_build_seconds(int32_t which, const int32_t* cu_seqlens_host, int32_t n_seqs, int32_t n_heads,
                                const hydra_pair_t* pairs, int32_t n_pairs, int32_t causal);
void hydra_shutdown(void);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif
#ifdef __cplusplus
}
#endif
#endif /* HYDRA_ATTN_H */
