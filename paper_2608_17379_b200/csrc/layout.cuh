// Memory layout of the attention tensors, shared by the forward and backward kernels.
//
// Two layouts are supported.  Packed (dense == 0): q, o, dout, dq are [T, Hq, D] and k, v, dk, dv are
// [T, Hkv, D]; sequence b owns the token rows cu_seqlens[b] .. cu_seqlens[b+1]-1; lse is [Hq, T].
// Dense (dense == 1): the tensors are [B, H, S, D] (the shape convention of the paper's attention
// workloads, appendix "Workloads"); sequence b owns rows 0 .. L_b-1 of its [H, S, D] block, with
// L_b = S, or cu_seqlens[b+1] - cu_seqlens[b] <= S when lengths are given; lse is [B, Hq, S].
// A row of either layout is addressed as (batch index, token, head): in the packed layout the batch
// index is 0 and the token is the global row, in the dense one the token is the position in the sequence.
// Workspace tensors of the backward pass (D_i, the fp32 dQ accumulator) are always indexed by the global
// token b * S + s (dense) or the packed row.
#pragma once
#include <stdint.h>

namespace sdpa {

struct TensorLayout {
    long long bs_q, bs_kv;  // batch strides in elements (unused in the packed layout)
    long long lse_bs;       // batch stride of lse
    int ts_q, hs_q;         // token and head stride of q, o, dout, dq in elements
    int ts_kv, hs_kv;       // token and head stride of k, v, dk, dv
    int lse_hs;             // head stride of lse
    int dense;              // 0 packed, 1 dense [B, H, S, D]
    int S;                  // dense: rows per sequence block
    int has_lengths;        // dense: cu_seqlens gives per-sequence lengths (else every sequence has S rows)
};

// Where sequence b starts.  tok0: first token coordinate of the sequence in the tensors; bidx: batch
// coordinate; gt0: first global token (workspace index); L: number of rows.  Returns false when
// cu_seqlens contradicts the launch parameters.
struct SeqPos {
    int tok0, bidx, gt0, L;
};
__device__ __forceinline__ bool locate_sequence(const TensorLayout& lay, const int32_t* cu_seqlens, int b, int T,
                                                int max_seqlen, SeqPos& sp) {
    if (lay.dense) {
        int L = lay.S;
        if (lay.has_lengths) {
            const int r0 = cu_seqlens[b], r1 = cu_seqlens[b + 1];
            L = r1 - r0;
            if (r0 < 0) return false;
        }
        if (L < 0 || L > lay.S || L > max_seqlen) return false;
        sp.tok0 = 0;
        sp.bidx = b;
        sp.gt0 = b * lay.S;
        sp.L = L;
        return true;
    }
    const int r0 = cu_seqlens[b], r1 = cu_seqlens[b + 1];
    const int L = r1 - r0;
    if (L < 0 || r0 < 0 || r1 > T || L > max_seqlen) return false;
    sp.tok0 = r0;
    sp.bidx = 0;
    sp.gt0 = r0;
    sp.L = L;
    return true;
}

// The tensor maps keep their strides increasing: dims {D, H, T, 1} for the packed layout, {D, S, H, B} for the
// dense one, so the token and head coordinates swap places between the two.
#define SDPA_TMA_LOAD_ROWS(dst, map, bar, d0, tok, head, bidx, dense)                       \
    tma_load_4d((dst), (map), (bar), (d0), (dense) ? (tok) : (head), (dense) ? (head) : (tok), (bidx))

}  // namespace sdpa
