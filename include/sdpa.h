/*
 * sdpa.h - C ABI of the B200 (sm_100a) bf16 scaled-dot-product-attention library.
 *
 * The primary pair is sdpa_fwd / sdpa_bwd over packed (variable-length) batches with grouped-query
 * heads; the other entry points are the same two passes for other layouts and shapes (dense
 * [B, H, S, D] tensors, separate key lengths, a paged KV cache, decode, a reproducible backward, host
 * buffers, built-in scratch) and the paper's bf16 GEMM.  Every step of the path runs in this library's
 * own CUDA kernels (TMA-staged tiles, tcgen05 MMAs with TMEM accumulators); there is no CPU path and
 * no call into any attention/GEMM library.
 *
 * Conventions shared by all entry points
 * --------------------------------------
 *  - All tensor pointers are DEVICE pointers, 16-byte aligned, contiguous, caller-owned.
 *    The library never allocates or frees memory; calls are asynchronous on `stream`
 *    (a cudaStream_t passed as void*, may be 0) and every buffer must stay alive until the
 *    stream has passed the call.
 *  - Token-major packed layout.  T = total_tokens = cu_seqlens[B].
 *        q, o, dout, dq : bf16 [T, Hq,  D]
 *        k, v, dk, dv   : bf16 [T, Hkv, D]
 *        lse            : fp32 [Hq, T]
 *        cu_seqlens     : int32 [B + 1] in device memory, cu_seqlens[0] = 0, non-decreasing;
 *                         sequence b owns token rows cu_seqlens[b] .. cu_seqlens[b+1]-1 of every
 *                         tensor (self-attention: queries and keys of a sequence have equal length).
 *  - Grouped-query attention: query head h reads kv head h / (Hq / Hkv).
 *  - causal != 0: query i of a sequence attends to keys 0..i of that sequence
 *    (lower-triangular mask); causal == 0: to all keys of its sequence.
 *  - Supported: D a multiple of 8 with 8 <= D <= 128 (the kernels are built for 64 and 128; another D
 *    runs in the next larger one with zero-padded columns, e.g. the paper's head dimension 96 at 3/4 of
 *    the arithmetic efficiency of 128; appendix "Workloads"); Hq a multiple of Hkv; scale finite and
 *    > 0; sequences of any length >= 0 (empty sequences and T = 0 are valid no-ops).
 *  - max_seqlen must be >= the longest sequence; total_tokens must equal cu_seqlens[B].  They
 *    size the launch grid and the TMA tensor maps without a device-to-host read of cu_seqlens.
 *    A cu_seqlens that contradicts them is reported through sdpa_query_status
 *    (SDPA_STATUS_BAD_CU_SEQLENS); outputs are then unspecified but no out-of-bounds access happens.
 *
 * Return value of the launching calls: SDPA_OK (0) when the work was enqueued, a negative
 * SDPA_ERR_* code when the call was rejected before any launch.  Problems found on the device
 * (a bounded wait that ran out, inconsistent cu_seqlens) are latched in a per-device status word
 * read by sdpa_query_status.
 */
#ifndef SDPA_B200_H_
#define SDPA_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SDPA_OK 0
#define SDPA_ERR_NULL (-1)      /* a required pointer is null */
#define SDPA_ERR_ALIGN (-2)     /* a tensor pointer is not 16-byte aligned */
#define SDPA_ERR_SHAPE (-3)     /* unsupported D, Hq % Hkv != 0, B < 1, negative sizes, bad scale */
#define SDPA_ERR_WORKSPACE (-4) /* workspace missing, misaligned or too small */
#define SDPA_ERR_ARCH (-5)      /* current device is not compute capability 10.x */
#define SDPA_ERR_CUDA (-6)      /* a CUDA runtime/driver call failed; see sdpa_last_cuda_error */
#define SDPA_ERR_STATIC_SCRATCH (-7) /* problem needs more than SDPA_STATIC_SCRATCH_BYTES of built-in scratch */

#define SDPA_STATUS_TIMEOUT 1        /* a device-side wait gave up; outputs of that call are invalid */
#define SDPA_STATUS_BAD_CU_SEQLENS 2 /* cu_seqlens / page table contradicts the sizes given, or breaks a length rule */
#define SDPA_STATUS_INTERNAL 3       /* a kernel found its own launch preconditions violated */

/*
 * Forward pass (paper, appendix "Workloads": MHA forward, causal and non-causal, returns a bf16
 * output and an fp32 log-sum-exp; "Generalization attention workloads": GQA over ragged batches;
 * evaluation order: the online-softmax tile loop of the corrected Algorithm 2, whose epilogue
 * defines O = diag(l)^-1 O and L = m + log l).
 *   o[r,h,:]  = sum_j softmax_j(scale * q[r,h,:] . k[j,g,:]) v[j,g,:]   over the allowed keys j
 *   lse[h,r]  = natural log of sum_j exp(scale * q[r,h,:] . k[j,g,:])   over the allowed keys j
 * q, k, v are read; o (bf16, round to nearest even) and lse (fp32) are overwritten for every
 * token row of every sequence.
 */
int sdpa_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
             const int32_t* cu_seqlens, int B, int Hq, int Hkv, int D, int causal, float scale,
             int total_tokens, int max_seqlen, void* stream);

/*
 * Forward pass over a paged KV cache (paper, appendix "Generalization attention workloads": GQA paged
 * causal prefill and paged decode, page size 1, key/value rows addressed through a list of page
 * indices; each returns a bf16 attention output and an fp32 log-sum-exp).
 *   q            : bf16 [total_q, Hq, D], packed by cu_seqlens_q (int32 [B+1], device)
 *   k_cache, v_cache : bf16 [num_pages, Hkv, D], one token per page
 *   kv_indptr    : int32 [B+1] (device); sequence b owns kv_indices[kv_indptr[b] .. kv_indptr[b+1]-1]
 *   kv_indices   : int32 page numbers in [0, num_pages), in key order
 *   o, lse       : as sdpa_fwd ([total_q, Hq, D] bf16, [Hq, total_q] fp32)
 * A sequence may have more keys than queries (Lk >= Lq, e.g. decode: Lq = 1).  With causal != 0 the
 * mask is aligned to the end: query i sees keys 0 .. i + (Lk - Lq); with causal == 0 all Lk keys.
 * A sequence with fewer keys than queries, or a page index outside [0, num_pages), is reported as
 * SDPA_STATUS_BAD_CU_SEQLENS (no out-of-range read happens).  Other conventions, supported D, return
 * codes: as sdpa_fwd.
 */
int sdpa_fwd_paged(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                   const int32_t* cu_seqlens_q, const int32_t* kv_indptr, const int32_t* kv_indices,
                   int B, int Hq, int Hkv, int D, int causal, float scale, int total_q,
                   int max_seqlen_q, int num_pages, void* stream);

/*
 * Bytes of scratch sdpa_bwd needs for these sizes (fp32 dQ accumulator [T,Hq,D] plus the fp32
 * row terms D_i [Hq,T]); 0 on invalid arguments.  The workspace must be 256-byte aligned device
 * memory; its contents on entry do not matter and are unspecified on exit.
 */
size_t sdpa_bwd_workspace_bytes(int B, int Hq, int Hkv, int D, int total_tokens, int max_seqlen);

/*
 * Backward pass (paper, appendix "Workloads": MHA backward consumes Q, K, V, the forward output,
 * its upstream gradient and the log-sum-exp, and returns bf16 gradients of Q, K, V).  With P
 * recomputed as exp(scale * q.k - lse):
 *   D_i = dout_i . o_i      dP = dout V^T      dS = P * (dP - D_i)
 *   dq = scale * dS K       dk = scale * dS^T Q       dv = P^T dout
 * dk and dv are summed over the Hq / Hkv query heads that share a kv head.  o and lse must be the
 * outputs of sdpa_fwd on the same q, k, v, cu_seqlens, causal and scale.  dq, dk, dv are
 * overwritten (not accumulated into).  dq partial sums from different key tiles are combined
 * with floating-point atomics, so dq may differ in the last bits from run to run.
 */
int sdpa_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse,
             const void* dout, void* dq, void* dk, void* dv, const int32_t* cu_seqlens, int B,
             int Hq, int Hkv, int D, int causal, float scale, int total_tokens, int max_seqlen,
             void* workspace, size_t workspace_bytes, void* stream);

/*
 * Decode over a paged KV cache (paper, appendix "Generalization attention workloads": GQA paged decode, one
 * query token per sequence, page size 1).  The same operator as sdpa_fwd_paged with one query row per
 * sequence, on a path built for that shape, which is bound by reading the K/V pages and not by arithmetic:
 * a CTA owns one (sequence, kv head) and one split of its keys, the rows of its tile are the Hq / Hkv query
 * heads of the group, so the group's pages are read once; a second small kernel merges the splits.
 *        q, o    : bf16 [B, Hq, D]            (token b is the query of sequence b)
 *        lse     : fp32 [Hq, B]
 *        k_cache, v_cache, kv_indptr, kv_indices, num_pages : as for sdpa_fwd_paged
 * The query sees all keys of its sequence; every sequence needs at least one key.  max_seqlen_k bounds the
 * key count of a sequence and fixes the number of key splits.  `workspace` is caller-owned, 256-byte
 * aligned device scratch of at least sdpa_decode_paged_workspace_bytes(...) bytes (fp32 partial results of
 * the splits).  Hq / Hkv must not exceed 128.  Errors and status reporting as for sdpa_fwd_paged.
 */
size_t sdpa_decode_paged_workspace_bytes(int B, int Hq, int Hkv, int D, int max_seqlen_k);
int sdpa_decode_paged(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                      const int32_t* kv_indptr, const int32_t* kv_indices, int B, int Hq, int Hkv, int D,
                      float scale, int max_seqlen_k, int num_pages, void* workspace,
                      size_t workspace_bytes, void* stream);

/*
 * Forward and backward passes for sequences whose keys are not the rows of their queries (the paper's paged
 * prefill workload has more keys than queries per sequence, appendix "Generalization attention workloads";
 * these are the same operator on packed tensors, with its backward pass):
 *        q, o, dout, dq : bf16 [total_q, Hq,  D]     rows of sequence b: cu_seqlens_q[b] .. cu_seqlens_q[b+1]-1
 *        k, v, dk, dv   : bf16 [total_k, Hkv, D]     rows of sequence b: cu_seqlens_k[b] .. cu_seqlens_k[b+1]-1
 *        lse            : fp32 [Hq, total_q]
 * causal != 0: query i of Lq attends to keys 0 .. i + (Lk - Lq) of its sequence (the last query sees the
 * last key), which needs Lk >= Lq; causal == 0: to all Lk keys, which needs Lk >= 1 wherever Lq >= 1.  A
 * sequence that breaks these rules is reported as SDPA_STATUS_BAD_CU_SEQLENS.  Keys of a sequence without
 * queries get zero dk and dv.  max_seqlen_q / max_seqlen_k bound the query / key lengths and size the
 * grids; the backward workspace is sdpa_bwd_workspace_bytes(B, Hq, Hkv, D, total_q, max_seqlen_q).
 * Everything else is as for sdpa_fwd / sdpa_bwd.
 */
int sdpa_fwd_varlen_qk(const void* q, const void* k, const void* v, void* o, float* lse,
                       const int32_t* cu_seqlens_q, const int32_t* cu_seqlens_k, int B, int Hq, int Hkv,
                       int D, int causal, float scale, int total_q, int total_k, int max_seqlen_q,
                       int max_seqlen_k, void* stream);
int sdpa_bwd_varlen_qk(const void* q, const void* k, const void* v, const void* o, const float* lse,
                       const void* dout, void* dq, void* dk, void* dv, const int32_t* cu_seqlens_q,
                       const int32_t* cu_seqlens_k, int B, int Hq, int Hkv, int D, int causal,
                       float scale, int total_q, int total_k, int max_seqlen_q, int max_seqlen_k,
                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * sdpa_bwd with a reproducible dq (the paper's backward workloads do not ask for this; the libraries it
 * compares with offer such a mode).  sdpa_bwd adds the dq contributions of the key tiles of a sequence
 * with fp32 reduce-adds in whatever order the tiles get there, so the last bits of dq can differ from run
 * to run (dk and dv never do).  This entry point makes the key tiles take turns on every 64-row block of
 * queries, from the highest key tile down, through per-block turn counters in the workspace: two calls on
 * the same inputs give bit-identical dq, dk, dv (dk and dv equal those of sdpa_bwd bit for bit).  Same
 * arguments, workspace size, errors and status reporting as sdpa_bwd.  It is slower because the key tiles
 * with the fewest visible queries have to be launched first instead of last (the tiles waited for must be
 * running already), which balances the SMs less well.  A turn wait is bounded like every other
 * device-side wait (SDPA_STATUS_TIMEOUT).
 */
int sdpa_bwd_deterministic(const void* q, const void* k, const void* v, const void* o, const float* lse,
                           const void* dout, void* dq, void* dk, void* dv, const int32_t* cu_seqlens,
                           int B, int Hq, int Hkv, int D, int causal, float scale, int total_tokens,
                           int max_seqlen, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same forward and backward passes on dense tensors in the shape convention of the paper's attention
 * workloads (appendix "Workloads": bf16 tensors of shape [batch, heads, sequence, head dim]):
 *        q, o, dout, dq : bf16 [B, Hq,  S, D]      k, v, dk, dv : bf16 [B, Hkv, S, D]
 *        lse            : fp32 [B, Hq, S]
 * all contiguous.  cu_seqlens may be null: every sequence then has S rows.  Otherwise it is the usual
 * int32 [B + 1] device array and sequence b uses rows 0 .. cu_seqlens[b+1] - cu_seqlens[b] - 1 (at most S)
 * of its [H, S, D] blocks.  Rows past a sequence's length never influence a result, but the tile loads
 * read them and multiply them by zero weights, so they must hold finite values (zeros, or anything left
 * by an earlier finite computation); in o, lse, dk and dv such rows are left untouched, in dq they are
 * written as zeros.  No transposed copy is made: the TMA tensor maps and the
 * stores walk the dense layout directly.  The backward workspace is sized by
 * sdpa_bwd_workspace_bytes(B, Hq, Hkv, D, B * S, S).  B * S must fit a 32-bit integer.  Everything else
 * (masking, GQA mapping, supported D, errors, status word) is as for sdpa_fwd / sdpa_bwd.
 */
int sdpa_fwd_bhsd(const void* q, const void* k, const void* v, void* o, float* lse,
                  const int32_t* cu_seqlens, int B, int Hq, int Hkv, int S, int D, int causal,
                  float scale, void* stream);
int sdpa_bwd_bhsd(const void* q, const void* k, const void* v, const void* o, const float* lse,
                  const void* dout, void* dq, void* dk, void* dv, const int32_t* cu_seqlens, int B,
                  int Hq, int Hkv, int S, int D, int causal, float scale, void* workspace,
                  size_t workspace_bytes, void* stream);

/*
 * Backward pass for callers that may not allocate device memory (the paper has no counterpart: this
 * is a convenience of this library, not one of its operators).
 *
 * sdpa_bwd needs scratch (the fp32 dQ accumulator and the D_i rows) that the caller normally
 * allocates.  Some callers cannot: a plug-in living inside a host runtime that hands out a fixed
 * arena at start-up and forbids cudaMalloc afterwards, a latency-critical loop in which the implicit
 * device synchronisation of an allocation is unacceptable, or code under a no-dynamic-allocation
 * rule after initialisation.  For them this entry point computes exactly what sdpa_bwd computes, with
 * the same arguments minus the workspace, and takes its scratch from a fixed array of
 * SDPA_STATIC_SCRATCH_BYTES (32 MiB) that is part of the library image: every GPU on which the
 * library is used holds these 32 MiB from the moment the library's module is loaded on it until the
 * process exits.  The call itself allocates and frees nothing (no cudaMalloc / cudaFree, no
 * allocating library routine); inputs and outputs are still caller-owned device buffers.
 *
 *  - Limit: sdpa_bwd_workspace_bytes(B, Hq, Hkv, D, total_tokens, max_seqlen) must not exceed
 *    SDPA_STATIC_SCRATCH_BYTES (about total_tokens * Hq * (D + 1) * 4 bytes; e.g. T*Hq <= 65,000
 *    at D = 128).  Larger problems are rejected with SDPA_ERR_STATIC_SCRATCH before anything is
 *    launched; use sdpa_bwd with your own workspace for those.
 *  - First use on a device: the first call made while a given device is current looks up the
 *    device address of the array (cudaGetSymbolAddress, once per device) before launching.  Make that
 *    first call during start-up, before any stream capture is begun on that device.
 *  - The array is shared by every call in the process and keeps whatever the previous call left in
 *    it.  Each call clears the part it accumulates into before using it, so calls that run one after
 *    the other on the GPU are independent; two calls that overlap on the GPU (different streams, or
 *    different host threads on different streams) race on the array and corrupt each other's dq.
 *    Serialise them, or give the concurrent ones sdpa_bwd with separate workspaces.
 * Errors and status reporting are those of sdpa_bwd.
 */
#define SDPA_STATIC_SCRATCH_BYTES (32u << 20)
int sdpa_bwd_static_scratch(const void* q, const void* k, const void* v, const void* o,
                            const float* lse, const void* dout, void* dq, void* dk, void* dv,
                            const int32_t* cu_seqlens, int B, int Hq, int Hkv, int D, int causal,
                            float scale, int total_tokens, int max_seqlen, void* stream);

/*
 * Whole step with HOST buffers (no counterpart in the paper's operator list beyond composing the
 * forward and backward workloads of its appendix "Workloads"): copies q, k, v, dout and cu_seqlens
 * from host memory to the device, runs sdpa_fwd then sdpa_bwd, and copies o, lse, dq, dk, dv back.
 * The work is ordered like any other work on `stream`: it starts after what was enqueued on `stream`
 * before the call, and what is enqueued on `stream` after the call starts when the host outputs are
 * complete; the host outputs are valid once the stream has been synchronised.  Inside, the step is cut
 * into up to four chunks of kv heads that are copied in, computed and copied out in a pipeline (compute
 * on `stream`, the copies on two internal non-blocking streams that fork from and join `stream` through
 * events), so that the two directions of the host link work at the same time.  The internal streams and
 * events are created on the calling thread's first call on a device (no device memory is allocated) and
 * kept.  Host pointers should be page-locked for the copies to overlap; layouts are those of sdpa_fwd /
 * sdpa_bwd.  `staging` is caller-owned, 256-byte aligned DEVICE scratch of at least
 * sdpa_host_staging_bytes(...) bytes that holds the device copies and the backward workspace.
 */
size_t sdpa_host_staging_bytes(int B, int Hq, int Hkv, int D, int total_tokens, int max_seqlen);
int sdpa_fwd_bwd_host(const void* q, const void* k, const void* v, const void* dout, void* o,
                      float* lse, void* dq, void* dk, void* dv, const int32_t* cu_seqlens, int B,
                      int Hq, int Hkv, int D, int causal, float scale, int total_tokens,
                      int max_seqlen, void* staging, size_t staging_bytes, void* stream);

/*
 * Profiling hook (measurement protocol of the paper's section "Multi-turn Evaluation Protocol":
 * per-kernel device timing): registers, for the calling thread, two caller-owned cudaEvent_t that
 * every later sdpa_bwd records on its stream immediately before and after its main kernel (between
 * the D_i preprocess and the dQ conversion).  Pass null pointers to switch it off.  Returns SDPA_OK.
 */
int sdpa_bwd_profile_events(void* ev_main_start, void* ev_main_stop);

/*
 * bf16 GEMM C = A B^T (paper, appendix "Workloads": the fifth primary workload, C = A B^T at BF16 with
 * A 8192x5120, B 7168x5120, C 8192x7168).  a [M,K], b [N,K], c [M,N]: row-major contiguous bf16
 * DEVICE pointers, 16-byte aligned, caller-owned; products are accumulated in fp32 on the tensor cores
 * and c is rounded to bf16 (nearest even) and overwritten.  Any M >= 0; N and K must be multiples of
 * 8 (16-byte row pitches), K > 0 unless the output is empty; other shapes return SDPA_ERR_SHAPE.
 * Asynchronous on `stream`; nothing is allocated.  Errors and the device status word are those of
 * the other entry points.
 */
int gemm_bf16_nt(const void* a, const void* b, void* c, int M, int N, int K, void* stream);

/*
 * Self-test of the failure path (the paper's profiling service isolates kernels that "may crash, hang,
 * or corrupt subsequent measurements", section "Multi-turn Evaluation Protocol"; this library instead
 * bounds every device-side wait).  Launches one warp that waits on a barrier nobody signals, with a
 * limit of `limit_cycles` SM cycles (1 .. 4e9).  The wait gives up, the kernel returns normally, and
 * the next sdpa_query_status reports SDPA_STATUS_TIMEOUT with site 99; the context stays usable.
 */
int sdpa_selftest_wait_timeout(long long limit_cycles, void* stream);

/*
 * Waits for `stream`, then returns the current device's status word (0 = no device-side problem
 * since the last query; otherwise an SDPA_STATUS_* code) and clears it.  *site (may be null)
 * receives an internal identifier of the wait that gave up.  Returns SDPA_ERR_CUDA if the
 * synchronisation or the copy failed.
 */
int sdpa_query_status(void* stream, int* site);

/* Static, human-readable name of a return or status code. */
const char* sdpa_status_string(int code);

/* The cudaError_t (as int) of the most recent failed runtime call made by this library on the
 * calling thread, or the CUresult of a failed tensor-map encode; 0 if none. */
int sdpa_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SDPA_B200_H_ */
