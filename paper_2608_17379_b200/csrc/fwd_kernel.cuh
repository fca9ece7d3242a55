// Forward attention kernel for sm_100a.
//
// One CTA owns two consecutive 128-row query tiles of one (sequence, query head) and walks the
// 128-row key/value tiles of that sequence.  Roles (warp-specialised, 12 warps):
//   warps 0-3   softmax group of query tile 0 (thread = one query row)
//   warps 4-7   softmax group of query tile 1
//   warp  8     MMA issuer (one elected lane): S = Q K^T and O += P V with tcgen05.mma
//   warp  9     TMA producer (one elected lane): Q tiles once, K/V tiles through an mbarrier ring
//   warps 10-11 idle (they complete the third warpgroup so registers can be re-balanced)
// TMEM (512 columns): S of tile 0 [0,128), S of tile 1 [128,256), O of tile 0 [256,256+D),
// O of tile 1 [384,384+D).  bf16 P overwrites the first 64 columns of its S and feeds the second
// MMA straight from TMEM.  While one group runs its softmax the tensor core works for the other.
//
// The loop is the online-softmax recurrence (running max m, running sum l, rescale of O when the
// max moves); O is only rescaled when the max grew by more than 2^8 in the exp2 domain, otherwise
// the stale max stays the reference, which changes nothing in exact arithmetic.
#pragma once
#include "ptx.cuh"
#include "layout.cuh"

#ifndef SDPA_TR
#define SDPA_TR(role, it, k) do { } while (0)
#endif

namespace sdpa {

struct FwdParams {
    const int32_t* cu_seqlens;   // query rows of sequence b: cu_seqlens[b] .. cu_seqlens[b+1]-1
    const int32_t* cu_seqlens_k; // key rows of sequence b in k / v (packed layout), or null: same rows as the queries
    int Tk;                      // rows of k / v when cu_seqlens_k is given
    // paged variant only: keys/values of sequence b are the cache rows kv_indices[kv_indptr[b] + j]
    const int32_t* kv_indptr;
    const int32_t* kv_indices;
    const __nv_bfloat16* k_cache;  // [num_pages, Hkv, D], page size 1
    const __nv_bfloat16* v_cache;
    int num_pages;
    __nv_bfloat16* o;
    float* lse;
    int* status;
    int B, Hq, Hkv, T;
    int causal;
    int max_seqlen;
    int d;             // head dimension of the tensors (multiple of 8, <= D of the kernel; columns d..D-1 are zero padding)
    TensorLayout lay;  // strides of q / o (and of k / v for the non-paged kernel), lse
    // decode variant only: per key split, unnormalised-free partial results of every (sequence, head)
    float* part_o;     // [2 * n_splits, B, Hq, d] fp32: softmax average of V over the keys of one slot of a split
    float* part_lse;   // [2 * n_splits, B, Hq] fp32: log-sum-exp over those keys (-inf where there were none)
    int tiles_per_split;  // decode variant: key tiles one CTA takes
    int head_chunk;    // (sequence, query head) pairs whose CTAs are launched interleaved
    float scale;       // softmax scale
    float scale_log2;  // scale * log2(e)
};

template <int D>
struct FwdCfg {
    static constexpr int kThreads = 384;
    static constexpr int kTile = 128;
    static constexpr int kTileBytes = kTile * D * 2;             // one Q, K or V tile
    static constexpr int kAtomBytes = kTile * 128;               // one 64-column swizzle atom of a tile
    static constexpr int kStages = (D == 128) ? 4 : 8;           // K/V ring slots
    static constexpr int kSmemQ = 2 * kTileBytes;
    static constexpr int kSmemRing = kStages * kTileBytes;
    static constexpr int kSmemBars = 1024;
    static constexpr int kSmemBytes = kSmemQ + kSmemRing + kSmemBars + 1024;  // + alignment slack
    static constexpr int kKSteps = D / 16;                       // k-steps of S = Q K^T
};

#ifndef SDPA_FWD_EMUL_PAIRS
#define SDPA_FWD_EMUL_PAIRS 2
#endif
constexpr int kEmulPairs = SDPA_FWD_EMUL_PAIRS;  // of every 8 score pairs, how many take the polynomial exp2

enum FwdSite {
    kSiteQFull = 1, kSiteKvFull = 2, kSiteKvEmpty = 3, kSiteSFull = 4, kSitePFull = 5, kSiteOFull = 6,
    kSiteDrain = 7
};

// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros instead of reading.
__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gsrc, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(src_bytes)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// kPaged = false: K/V are tensors loaded by TMA; the keys of a sequence are the rows of its queries, or (packed
// layout, cu_seqlens_k given) a row range of their own.  kPaged = true: K/V rows are gathered from a
// page-size-1 cache through a page table.  Whenever a sequence has Lk keys for Lq queries, a causal query i
// sees keys 0 .. i + (Lk - Lq): the last query sees the last key.
template <int D, bool kPaged, bool kDecode = false>
__global__ void __launch_bounds__(384, 1)
sdpa_fwd_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const FwdParams p) {
    using Cfg = FwdCfg<D>;
    // ring slots; the decode variant has no second Q tile and adds that buffer to the ring
    constexpr int S = kDecode ? Cfg::kStages + 1 : Cfg::kStages;

    static_assert(!kDecode || kPaged, "the decode variant reads a paged cache");
    int b, h, g, r0, L, q_start;
    SeqPos sp;
    if (kDecode) {
        // Decode: one query token per sequence.  A CTA owns one (sequence, kv head) and one split of its keys;
        // the rows of its single query tile are the G query heads of the group (GQA packing), so the group's
        // K/V rows are gathered once and not once per head.  grid = (B * Hkv, key splits).
        const int bg = blockIdx.x;
        b = bg / p.Hkv;
        g = bg % p.Hkv;
        h = g * (p.Hq / p.Hkv);  // first query head of the group
        sp.tok0 = b; sp.bidx = 0; sp.gt0 = b; sp.L = 1;
        r0 = b;
        L = 1;
        q_start = 0;
    } else {
        // Launch order: the (sequence, query head) pairs are taken in chunks of p.head_chunk; inside a chunk
        // the CTAs go query-tile pair by pair (heaviest first), chunk after chunk, so the K/V rows that the
        // CTAs running at one time walk through fit the L2 (the host picks the chunk from the K/V size per head).
        const int bh = (int)blockIdx.y * p.head_chunk + (int)blockIdx.x % p.head_chunk;
        if (bh >= p.B * p.Hq) return;
        const int pair_raw = (int)blockIdx.x / p.head_chunk;
        const int n_pairs_grid = (int)gridDim.x / p.head_chunk;
        b = bh / p.Hq;
        h = bh % p.Hq;
        g = h / (p.Hq / p.Hkv);
        const int pair = n_pairs_grid - 1 - pair_raw;  // heaviest (latest) query tiles first
        if (!locate_sequence(p.lay, p.cu_seqlens, b, p.T, p.max_seqlen, sp)) {
            if (threadIdx.x == 0) atomicCAS(p.status, 0, kStatusBadCuSeqlens);
            return;
        }
        r0 = sp.tok0;  // token coordinate of the sequence's first row
        L = sp.L;
        q_start = pair * 256;
        if (q_start >= L) return;
    }
    const int G = p.Hq / p.Hkv;
    int Lk = L, kbase = 0;  // number of keys of this sequence; first entry of its page list
    if (kPaged) {
        kbase = p.kv_indptr[b];
        Lk = p.kv_indptr[b + 1] - kbase;
        if (Lk < L || kbase < 0) {  // fewer keys than queries would leave fully masked rows
            if (threadIdx.x == 0) atomicCAS(p.status, 0, kStatusBadCuSeqlens);
            return;
        }
    }
    int rk0 = r0;  // first key row of the sequence in k / v
    if (!kPaged && p.cu_seqlens_k != nullptr) {
        rk0 = p.cu_seqlens_k[b];
        const int rk1 = p.cu_seqlens_k[b + 1];
        Lk = rk1 - rk0;
        // every query row needs a visible key: at least one key, and under the end-aligned causal mask at
        // least as many keys as queries
        if (rk0 < 0 || rk1 > p.Tk || Lk < 1 || (p.causal && Lk < L)) {
            if (threadIdx.x == 0) atomicCAS(p.status, 0, kStatusBadCuSeqlens);
            return;
        }
    }
    const int off = Lk - L;  // causal alignment: the last query sees the last key

    int n_kv[2];
    const int n_kv_all = (Lk + 127) >> 7;
    int tile_begin = 0;  // first key tile of this CTA (decode: the start of its split)
    if (kDecode) {
        const int per_split = p.tiles_per_split;  // key tiles per CTA, the same for every sequence
        tile_begin = (int)blockIdx.y * per_split;
        const int n_mine = min(n_kv_all, tile_begin + per_split) - tile_begin;
        // The two tile slots of the CTA work on the same query rows and take the split's key tiles in turn
        // (slot t: tiles t, t+2, ...), each with its own running maximum, sum and accumulator, so that one
        // slot's softmax overlaps the other's MMAs; they leave two partial results for the combining kernel.
        n_kv[0] = max(0, (n_mine + 1) >> 1);
        n_kv[1] = max(0, n_mine >> 1);
        if (n_mine <= 0) {  // nothing in this split: the combining kernel skips a partial whose lse is -inf
            if ((int)threadIdx.x < 2 * G)
                p.part_lse[(static_cast<size_t>(2 * blockIdx.y + threadIdx.x / G) * p.B + b) * p.Hq + h + threadIdx.x % G] =
                    -INFINITY;
            return;
        }
    } else {
        const bool has1 = (q_start + 128) < L;
        n_kv[0] = p.causal ? min(n_kv_all, ((q_start + 127 + off) >> 7) + 1) : n_kv_all;
        n_kv[1] = has1 ? (p.causal ? min(n_kv_all, ((q_start + 255 + off) >> 7) + 1) : n_kv_all) : 0;
    }
    const int n_iter = kDecode ? n_kv[0] + n_kv[1] : max(n_kv[0], n_kv[1]);  // decode: key tiles of the CTA

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;
    uint8_t* sRing = kDecode ? sQ + Cfg::kTileBytes : smem + Cfg::kSmemQ;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kSmemQ + Cfg::kSmemRing);
    uint64_t* q_full = bars;               // [2]
    uint64_t* kv_full = bars + 2;          // [S]
    uint64_t* kv_empty = bars + 2 + S;     // [S]
    uint64_t* s_full = bars + 2 + 2 * S;   // [2]
    uint64_t* p_full = s_full + 2;         // [2]
    uint64_t* o_full = p_full + 2;         // [2]
    uint64_t* drain = o_full + 2;          // [1]
    uint64_t* p_half = drain + 1;          // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(p_half + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const WaitCtl ctl{p.status, abort_flag};

    if (tid == 0) {
        *abort_flag = 0;
        for (int i = 0; i < 2; ++i) {
            mbar_init(&q_full[i], 1);
            mbar_init(&s_full[i], 1);
            // decode: only the warps that own query heads (rows below G) take part in the softmax hand-shake
            const int p_count = kDecode ? 32 * ((G + 31) / 32) : 128;
            mbar_init(&p_full[i], p_count);
            mbar_init(&p_half[i], p_count);
            mbar_init(&o_full[i], 1);
        }
        for (int i = 0; i < S; ++i) {
            mbar_init(&kv_full[i], kPaged ? 32 : 1);  // TMA transaction, or the 32 gathering lanes
            mbar_init(&kv_empty[i], 1);
        }
        mbar_init(drain, 1);
        fence_mbar_init();
    }
    if (warp == 8) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    if (warp == 9 && elect_one()) {
        prefetch_tmap(&map_q);
        prefetch_tmap(&map_k);
        prefetch_tmap(&map_v);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // ------------------------------------------------------------ gathering producers (paged variants)
    // Warps 9-11; in the decode variant also the softmax warps that own no query head.
    // A gatherer's next item is n_gather items ahead; with more gatherers than ring slots it could run two
    // revolutions of the ring ahead of the consumer, which the one-bit phase of an mbarrier cannot tell from
    // one revolution (seen as a corrupted ring and a wait that ran out).  So at most S warps gather.
    const int n_live = kDecode ? 2 * ((G + 31) / 32) : 8;  // softmax warps that do arithmetic
    const int n_gather = min(3 + (8 - n_live), S);
    auto gather_role = [&](int pw) {
            // -------------------------------------------------------- gathering producers (warps 9-11, all lanes)
            // K_j is ring item 2j, V_j item 2j+1; item `it` is gathered by gathering warp it % n_gather, so several
            // tiles are in flight.  A tile's 128 rows come from the page-size-1 cache with 16-byte cp.async into the same
            // 128B-swizzled layout a TMA load would produce; D/8 consecutive lanes copy one row (full lines in
            // the cache), the page numbers travel by shuffle.  Rows past the sequence end and the padding
            // columns are zero-filled (a masked P of exactly 0 must not meet garbage in V).
            const int lane = tid & 31;
            if (pw == 0 && lane == 0) {
                // decode: the Q map's box is the G heads of the group for one token (G rows of the tile)
                mbar_arrive_expect_tx(&q_full[0], kDecode ? static_cast<uint32_t>(G) * D * 2u : Cfg::kTileBytes);
#pragma unroll
                for (int a = 0; a < D / 64; ++a)
                    SDPA_TMA_LOAD_ROWS(sQ + a * Cfg::kAtomBytes, &map_q, &q_full[0], a * 64, r0 + q_start, h, sp.bidx, p.lay.dense);
                if (!kDecode && n_kv[1] > 0) {  // decode: both slots read the one Q tile
                    mbar_arrive_expect_tx(&q_full[1], Cfg::kTileBytes);
#pragma unroll
                    for (int a = 0; a < D / 64; ++a)
                        SDPA_TMA_LOAD_ROWS(sQ + Cfg::kTileBytes + a * Cfg::kAtomBytes, &map_q, &q_full[1], a * 64,
                                    r0 + q_start + 128, h, sp.bidx, p.lay.dense);
                }
            }
            constexpr int kLanesPerRow = D / 8;               // 16-byte chunks of a row
            constexpr int kRowsPerCopy = 32 / kLanesPerRow;    // rows one warp-wide cp.async covers
            const int my_c = lane % kLanesPerRow;
            const int my_sub = lane / kLanesPerRow;
            bool ok = true;
            for (int it = pw; it < 2 * n_iter && ok; it += n_gather) {
                // which tile ring item `it` is: K_0 V_0 K_1 V_1 ... in general; the decode variant consumes
                // K_0 K_1 V_0 K_2 V_1 K_3 ... V_(n-2) V_(n-1) (two slots, each one tile ahead with its S)
                int j = it >> 1, kv = it & 1;
                if (kDecode) {
                    if (it == 0) { j = 0; kv = 0; }
                    else if (it == 1 && n_iter > 1) { j = 1; kv = 0; }
                    else if (it <= 2 * n_iter - 3) { kv = (it & 1) ^ 1; j = kv ? (it - 2) >> 1 : (it + 1) >> 1; }
                    else { kv = 1; j = it - n_iter; }
                }
                // cache row addresses of the rows lane, lane+32, lane+64, lane+96 of key tile j (0: past the end)
                const __nv_bfloat16* cache = kv == 0 ? p.k_cache : p.v_cache;
                unsigned long long row_ptr[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int key = (tile_begin + j) * 128 + lane + 32 * i;
                    unsigned long long ptr = 0ull;
                    if (key < Lk) {
                        const int pg = p.kv_indices[kbase + key];
                        if (pg < 0 || pg >= p.num_pages)  // never read outside the cache
                            atomicCAS(p.status, 0, kStatusBadCuSeqlens);
                        else
                            ptr = reinterpret_cast<unsigned long long>(cache + (static_cast<size_t>(pg) * p.Hkv + g) * p.d);
                    }
                    row_ptr[i] = ptr;
                }
                const int st = it % S;
                ok = mbar_wait_warp(&kv_empty[st], ((it / S) & 1) ^ 1, ctl, kSiteKvEmpty);
                if (!ok) break;
                // Per copy only the row address (two shuffles) and a constant XOR change: the lane's column
                // chunk, its sub-row and the swizzle term they give are fixed.  row & 7 = (rr & 7) | my_sub
                // because rr is a multiple of the rows per copy, so chunk ^ (row & 7) = (chunk ^ my_sub) ^ (rr & 7).
                const bool col_real = my_c * 8 < p.d;
                const uint32_t dst_lane = smem_u32(sRing + st * Cfg::kTileBytes) + (my_c >> 3) * Cfg::kAtomBytes + my_sub * 128;
                const uint32_t swz_lane = static_cast<uint32_t>((my_c & 7) ^ my_sub);
                const unsigned long long col_off = static_cast<unsigned long long>(my_c) * 16ull;
#pragma unroll
                for (int rr = 0; rr < 128; rr += kRowsPerCopy) {
                    const unsigned long long base = __shfl_sync(0xffffffffu, row_ptr[rr >> 5], (rr + my_sub) & 31);
                    const bool real = base != 0ull && col_real;
                    const uint32_t dst = dst_lane + rr * 128 + ((swz_lane ^ (rr & 7)) << 4);
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst),
                                 "l"(real ? base + col_off : reinterpret_cast<unsigned long long>(cache)), "r"(real ? 16u : 0u)
                                 : "memory");
                }
                cp_async_commit();
                // The item is handed over before this warp asks for its next slot: that slot is freed by MMAs
                // which may themselves be waiting for this item.  The overlap comes from the other two warps.
                cp_async_wait<0>();          // the copies have landed
                fence_proxy_async_smem();    // make them visible to the tensor core's reads
                mbar_arrive(&kv_full[st]);
            }
            cp_async_wait<0>();
    };

    if (warp < 8) {
        // ------------------------------------------------------------ softmax groups
        setmaxnreg_inc<208>();
        const int t = warp >> 2;                 // which query tile
        const int row_in_tile = tid & 127;
        const int row = q_start + t * 128 + row_in_tile;  // row inside the sequence
        const bool valid = kDecode ? row_in_tile < G : row < L;
        // decode: only the first G rows of the tile are query heads; warps that own none of them do no
        // arithmetic and only keep the barriers in step
        const bool warp_live = !kDecode || (warp & 3) * 32 < G;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_base + t * 128;
        const uint32_t tO = tmem + lane_base + 256 + t * 128;
        float m = -INFINITY, l = 0.f;
        const int n = n_kv[t];
        bool ok = true;
        if (kPaged && !warp_live) {
            // decode: this warp owns no query head; it gathers K/V tiles instead (gatherers 3, 4, ...)
            const int live_per_group = (G + 31) / 32;
            const int pw = 3 + t * (4 - live_per_group) + ((warp & 3) - live_per_group);
            if (pw < n_gather) gather_role(pw);
            ok = false;  // nothing to store
        }
        for (int j = 0; j < n && ok; ++j) {
            if (row_in_tile == 0) SDPA_TR(t, j, 0);
            ok = mbar_wait_warp(&s_full[t], j & 1, ctl, kSiteSFull);
            if (!ok) break;
            if (row_in_tile == 0) SDPA_TR(t, j, 1);
            tc_fence_after();
            float s[128];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t r[32];
                tmem_ld_x32(tS + c * 32, r);
#pragma unroll
                for (int i = 0; i < 32; ++i) s[c * 32 + i] = __uint_as_float(r[i]);
            }
            tmem_wait_ld();
            if (row_in_tile == 0) SDPA_TR(t, j, 2);
            if (kDecode && !valid) {  // rows past the group's heads hold whatever was in shared memory: neutralise them
#pragma unroll
                for (int c = 0; c < 128; ++c) s[c] = 0.f;
            }
            const int key0 = (tile_begin + (kDecode ? 2 * j + t : j)) * 128;
            const bool diag = p.causal && (key0 + 127 > q_start + t * 128 + off);
            if (diag || key0 + 128 > Lk) {
                const int lim = p.causal ? min(row + off, Lk - 1) : (Lk - 1);  // last allowed key
#pragma unroll
                for (int c = 0; c < 128; ++c)
                    if (key0 + c > lim) s[c] = -INFINITY;
            }
            float mx0 = s[0], mx1 = s[1], mx2 = s[2], mx3 = s[3];
#pragma unroll
            for (int c = 4; c < 124; c += 8) {
                mx0 = max3(mx0, s[c], s[c + 1]);
                mx1 = max3(mx1, s[c + 2], s[c + 3]);
                mx2 = max3(mx2, s[c + 4], s[c + 5]);
                mx3 = max3(mx3, s[c + 6], s[c + 7]);
            }
            mx0 = max3(mx0, s[124], s[125]);
            mx1 = max3(mx1, s[126], s[127]);
            const float mx = fmaxf(max3(mx0, mx1, mx2), mx3);
            if (j == 0) {
                m = mx;
            } else {
                const bool grow = (mx - m) * p.scale_log2 > 8.0f;
                if (__any_sync(0xffffffffu, grow)) {
                    const float m_new = fmaxf(m, mx);
                    const float alpha = fast_exp2((m - m_new) * p.scale_log2);
                    m = m_new;
                    l *= alpha;
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t r[32];
                        tmem_ld_x32(tO + c * 32, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                        tmem_st_x32(tO + c * 32, r);
                    }
                }
            }
            if (row_in_tile == 0) SDPA_TR(t, j, 3);
            // p = exp2(s * c - m * c) on pairs of scores: one packed FMA, then either two SFU ex2 or (for
            // kEmulPairs of every eight pairs) the FMA-pipe polynomial, so the SFU is not the only exp unit.
            const float neg_m = -m * p.scale_log2;
            const uint64_t c2 = pack_f32x2(p.scale_log2, p.scale_log2), nm2 = pack_f32x2(neg_m, neg_m);
            uint64_t sum_a = pack_f32x2(0.f, 0.f), sum_b = pack_f32x2(0.f, 0.f);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t r[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const uint64_t x2 = fma_f32x2(pack_f32x2(s[c * 64 + 2 * i], s[c * 64 + 2 * i + 1]), c2, nm2);
                    uint64_t e2;
                    if ((i & 7) < kEmulPairs) {
                        e2 = exp2_poly_x2(x2);
                    } else {
                        float x0, x1;
                        unpack_f32x2(x2, x0, x1);
                        e2 = pack_f32x2(fast_exp2(x0), fast_exp2(x1));
                    }
                    if (i & 1) sum_b = add_f32x2(sum_b, e2);
                    else sum_a = add_f32x2(sum_a, e2);
                    float e0, e1;
                    unpack_f32x2(e2, e0, e1);
                    r[i] = pack_bf16x2(e0, e1);
                }
                tmem_st_x32(tS + c * 32, r);
                if (c == 0) {
                    // the first 64 keys of P are complete: P V may start on them while the rest is computed
                    tmem_wait_st();
                    tc_fence_before();
                    mbar_arrive(&p_half[t]);
                }
            }
            {
                float a0, a1, b0, b1;
                unpack_f32x2(sum_a, a0, a1);
                unpack_f32x2(sum_b, b0, b1);
                l += (a0 + a1) + (b0 + b1);
            }
            if (row_in_tile == 0) SDPA_TR(t, j, 4);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&p_full[t]);
            if (row_in_tile == 0) SDPA_TR(t, j, 5);
        }
        if (ok && n > 0) ok = mbar_wait_warp(&o_full[t], 0, ctl, kSiteOFull);
        if (kDecode) {
            // the G rows of the group leave as fp32 partial results of this key split
            const size_t slot = (static_cast<size_t>(2 * blockIdx.y + t) * p.B + b) * p.Hq + h + row_in_tile;
            if (n == 0 && valid) p.part_lse[slot] = -INFINITY;  // this slot had no key tile
            if (ok && n > 0 && warp_live) {
                tc_fence_after();
                const float inv_l = 1.0f / l;
                float* dst = p.part_o + slot * p.d;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld_x32(tO + c * 32, r);
                    tmem_wait_ld();
                    if (valid) {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if (c * 32 + i * 4 < p.d)
                                *reinterpret_cast<float4*>(dst + c * 32 + i * 4) =
                                    make_float4(__uint_as_float(r[4 * i]) * inv_l, __uint_as_float(r[4 * i + 1]) * inv_l,
                                                __uint_as_float(r[4 * i + 2]) * inv_l, __uint_as_float(r[4 * i + 3]) * inv_l);
                    }
                }
                if (valid) p.part_lse[slot] = m * p.scale + logf(l);
            }
        } else if (ok && n > 0) {
            tc_fence_after();
            const float inv_l = 1.0f / l;
            // O leaves through this tile's Q buffer (dead after the last S = Q K^T): every thread writes its
            // normalised bf16 row there (16-byte chunks XOR-swizzled by row so the writes spread over the
            // banks), then each warp copies its own 32 rows out with full-line stores.  Storing the rows
            // straight from the TMEM layout (thread = row) would touch 32 different lines per store.
            constexpr int kChunks = D / 8;             // 16-byte chunks per row
            constexpr int kRowsPerPass = 32 / kChunks;  // rows one warp store covers
            uint8_t* stage = sQ + t * Cfg::kTileBytes;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                tmem_ld_x32(tO + c * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 w;
                    w.x = pack_bf16x2(__uint_as_float(r[8 * i + 0]) * inv_l, __uint_as_float(r[8 * i + 1]) * inv_l);
                    w.y = pack_bf16x2(__uint_as_float(r[8 * i + 2]) * inv_l, __uint_as_float(r[8 * i + 3]) * inv_l);
                    w.z = pack_bf16x2(__uint_as_float(r[8 * i + 4]) * inv_l, __uint_as_float(r[8 * i + 5]) * inv_l);
                    w.w = pack_bf16x2(__uint_as_float(r[8 * i + 6]) * inv_l, __uint_as_float(r[8 * i + 7]) * inv_l);
                    const int k = c * 4 + i;
                    *reinterpret_cast<uint4*>(stage + row_in_tile * (D * 2) + ((k ^ (row_in_tile & 7)) << 4)) = w;
                }
            }
            __syncwarp();
            {
                const int lane = tid & 31;
                const int k = lane % kChunks;
                const int rows_left = L - (q_start + t * 128);  // rows of this tile inside the sequence
#pragma unroll
                for (int pass = 0; pass < 32 / kRowsPerPass; ++pass) {
                    const int rr = (warp & 3) * 32 + pass * kRowsPerPass + lane / kChunks;  // row inside the tile
                    if (rr < rows_left && k * 8 < p.d) {
                        const uint4 w = *reinterpret_cast<const uint4*>(stage + rr * (D * 2) + ((k ^ (rr & 7)) << 4));
                        __nv_bfloat16* dst = p.o + sp.bidx * p.lay.bs_q +
                                             static_cast<long long>(r0 + q_start + t * 128 + rr) * p.lay.ts_q +
                                             static_cast<long long>(h) * p.lay.hs_q;
                        *reinterpret_cast<uint4*>(dst + k * 8) = w;
                    }
                }
            }
            if (valid)
                p.lse[sp.bidx * p.lay.lse_bs + static_cast<long long>(h) * p.lay.lse_hs + r0 + row] = m * p.scale + logf(l);
        }
    } else {
        setmaxnreg_dec<80>();
        if (warp >= 9 && kPaged) {
            gather_role(warp - 9);
        } else if (warp == 9) {
            // -------------------------------------------------------- TMA producer
            if (elect_one()) {
                int it = 0;
                auto load_tile = [&](const CUtensorMap* map, uint8_t* dst, uint64_t* bar, int head, int tok) {
                    mbar_arrive_expect_tx(bar, Cfg::kTileBytes);
#pragma unroll
                    for (int a = 0; a < D / 64; ++a)
                        SDPA_TMA_LOAD_ROWS(dst + a * Cfg::kAtomBytes, map, bar, a * 64, tok, head, sp.bidx, p.lay.dense);
                };
                bool ok = true;
                load_tile(&map_q, sQ, &q_full[0], h, r0 + q_start);
                for (int j = 0; j < n_iter && ok; ++j) {
                    for (int kv = 0; kv < 2 && ok; ++kv, ++it) {
                        const int st = it % S;
                        ok = mbar_wait(&kv_empty[st], ((it / S) & 1) ^ 1, ctl, kSiteKvEmpty);
                        if (!ok) break;
                        load_tile(kv == 0 ? &map_k : &map_v, sRing + st * Cfg::kTileBytes, &kv_full[st], g,
                                  rk0 + j * 128);
                        if (j == 0 && kv == 0 && n_kv[1] > 0)
                            load_tile(&map_q, sQ + Cfg::kTileBytes, &q_full[1], h, r0 + q_start + 128);
                    }
                }
                if (!ok) {
                    // abandon: let the copies already issued land before the CTA exits
                    for (int back = 1; back <= S && back <= it; ++back) {
                        const int i2 = it - back;
                        mbar_wait(&kv_full[i2 % S], (i2 / S) & 1, ctl, kSiteDrain);
                    }
                }
            }
        } else if (warp == 8) {
            // -------------------------------------------------------- MMA issuer
            if (elect_one()) {
                constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, false, false);
                constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, false, true);
                // The issuing thread's own instruction stream bounds the MMA rate (every extra ALU
                // instruction between two tcgen05.mma costs several cycles), so descriptors are built
                // once and only advanced by constants inside the loops.
                const uint64_t q_desc0 = smem_desc_sw128(smem_u32(sQ), 0, 1024);
                const uint64_t q_desc1 = smem_desc_sw128(smem_u32(sQ) + Cfg::kTileBytes, 0, 1024);
                const uint64_t k_desc = smem_desc_sw128(smem_u32(sRing), 0, 1024);                 // K-major
                const uint64_t v_desc = smem_desc_sw128(smem_u32(sRing), Cfg::kAtomBytes, 1024);  // MN-major
                auto issue_qk = [&](int t, int st) {
                    const uint64_t a0 = t == 0 ? q_desc0 : q_desc1;
                    const uint64_t b0 = k_desc + static_cast<uint64_t>(st * (Cfg::kTileBytes >> 4));
                    const uint32_t d = tmem + t * 128;
#pragma unroll
                    for (int kk = 0; kk < Cfg::kKSteps; ++kk) {
                        const uint64_t off = static_cast<uint64_t>(((kk >> 2) * Cfg::kAtomBytes + (kk & 3) * 32) >> 4);
                        umma_ss(d, a0 + off, b0 + off, idesc_qk, kk > 0);
                    }
                };
                auto issue_pv = [&](int t, int st, bool accumulate, int half) {
                    const uint64_t b0 = v_desc + static_cast<uint64_t>(st * (Cfg::kTileBytes >> 4));
                    const uint32_t d = tmem + 256 + t * 128;
                    const uint32_t a = tmem + t * 128;
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4) {
                        const int kk = half * 4 + k4;
                        umma_ts(d, a + kk * 8, b0 + static_cast<uint64_t>(kk * (2048 >> 4)), idesc_pv,
                                (accumulate || kk > 0) ? 1u : 0u);
                    }
                };
                bool ok = true;
                int it = 0;  // ring consumer counter: K_j is item 2j, V_j is item 2j+1
                if (kDecode) {
                    // two slots on the same query rows (both use Q tile 0), slot t takes key tiles t, t+2, ...
                    const int n = n_iter;
                    auto next_item = [&]() {
                        const int st = it % S;
                        const bool w = mbar_wait(&kv_full[st], (it / S) & 1, ctl, kSiteKvFull);
                        ++it;
                        if (w) tc_fence_after();
                        ok = w;
                        return st;
                    };
                    auto issue_qk0 = [&](int t, int st) {
                        const uint64_t b0 = k_desc + static_cast<uint64_t>(st * (Cfg::kTileBytes >> 4));
                        const uint32_t d = tmem + t * 128;
#pragma unroll
                        for (int kk = 0; kk < Cfg::kKSteps; ++kk) {
                            const uint64_t off = static_cast<uint64_t>(((kk >> 2) * Cfg::kAtomBytes + (kk & 3) * 32) >> 4);
                            umma_ss(d, q_desc0 + off, b0 + off, idesc_qk, kk > 0);
                        }
                    };
                    ok = mbar_wait(&q_full[0], 0, ctl, kSiteQFull);
                    for (int t = 0; t < 2 && t < n && ok; ++t) {
                        const int st = next_item();
                        if (!ok) break;
                        issue_qk0(t, st);
                        umma_commit(&s_full[t]);
                        umma_commit(&kv_empty[st]);
                    }
                    for (int j = 0; j < n && ok; ++j) {
                        const int t = j & 1, i = j >> 1;
                        const int st_v = next_item();
                        if (!ok) break;
                        ok = mbar_wait(&p_half[t], i & 1, ctl, kSitePFull);
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv(t, st_v, i > 0, 0);
                        ok = mbar_wait(&p_full[t], i & 1, ctl, kSitePFull);
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv(t, st_v, i > 0, 1);
                        umma_commit(&kv_empty[st_v]);
                        if (j + 2 < n) {
                            const int st_k = next_item();
                            if (!ok) break;
                            issue_qk0(t, st_k);
                            umma_commit(&s_full[t]);
                            umma_commit(&kv_empty[st_k]);
                        } else {
                            umma_commit(&o_full[t]);
                        }
                    }
                    if (!ok) {
                        umma_commit(drain);
                        mbar_wait(drain, 0, ctl, kSiteDrain);
                    }
                    goto mma_done;
                }
                ok = mbar_wait(&q_full[0], 0, ctl, kSiteQFull);
                if (ok) ok = mbar_wait(&kv_full[0], 0, ctl, kSiteKvFull);
                if (ok) {
                    tc_fence_after();
                    issue_qk(0, 0);
                    umma_commit(&s_full[0]);
                    if (n_kv[1] > 0) {
                        ok = mbar_wait(&q_full[1], 0, ctl, kSiteQFull);
                        if (ok) {
                            tc_fence_after();
                            issue_qk(1, 0);
                            umma_commit(&s_full[1]);
                        }
                    }
                    umma_commit(&kv_empty[0]);
                    it = 1;
                }
                for (int j = 0; j < n_iter && ok; ++j) {
                    const int st_v = it % S;
                    SDPA_TR(2, j, 0);
                    ok = mbar_wait(&kv_full[st_v], (it / S) & 1, ctl, kSiteKvFull);
                    if (!ok) break;
                    SDPA_TR(2, j, 1);
                    ++it;
                    const bool have_next = (j + 1) < n_iter;
                    const int st_k = it % S;
                    bool next_ready = false;
                    for (int t = 0; t < 2 && ok; ++t) {
                        if (j >= n_kv[t]) continue;
                        ok = mbar_wait(&p_half[t], j & 1, ctl, kSitePFull);
                        if (!ok) break;
                        SDPA_TR(2, j, 2 + 2 * t);
                        tc_fence_after();
                        issue_pv(t, st_v, j > 0, 0);
                        ok = mbar_wait(&p_full[t], j & 1, ctl, kSitePFull);
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv(t, st_v, j > 0, 1);
                        if (j + 1 < n_kv[t]) {
                            if (!next_ready) {
                                ok = mbar_wait(&kv_full[st_k], (it / S) & 1, ctl, kSiteKvFull);
                                if (!ok) break;
                                tc_fence_after();
                                next_ready = true;
                            }
                            issue_qk(t, st_k);
                            umma_commit(&s_full[t]);
                        } else {
                            umma_commit(&o_full[t]);
                        }
                        SDPA_TR(2, j, 3 + 2 * t);
                    }
                    if (!ok) break;
                    umma_commit(&kv_empty[st_v]);
                    if (have_next) {
                        umma_commit(&kv_empty[st_k]);
                        ++it;
                    }
                }
                if (!ok) {
                    // abandon: wait (bounded) until the MMAs already issued have left the pipe
                    umma_commit(drain);
                    mbar_wait(drain, 0, ctl, kSiteDrain);
                }
            mma_done:;
            }
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem, 512);
}

// Decode, second step: merges the key splits of every (sequence, head).  With lse_s the log-sum-exp and o_s
// the softmax average of split s:  lse = log sum_s exp(lse_s),  o = sum_s exp(lse_s - lse) o_s.
// One CTA per (sequence, head), one thread per 4 columns.
__global__ void __launch_bounds__(32)
sdpa_decode_combine_kernel(const float* __restrict__ part_o, const float* __restrict__ part_lse,
                           __nv_bfloat16* __restrict__ o, float* __restrict__ lse, int n_splits, int B, int Hq, int d) {
    const int bh = blockIdx.x;  // b * Hq + h
    const int b = bh / Hq, h = bh % Hq;
    const size_t stride = static_cast<size_t>(B) * Hq;
    float mx = -INFINITY;
    for (int s = 0; s < n_splits; ++s) mx = fmaxf(mx, part_lse[s * stride + bh]);
    float sum = 0.f;
    for (int s = 0; s < n_splits; ++s) sum += expf(part_lse[s * stride + bh] - mx);
    const float total = mx + logf(sum);
    const int c = threadIdx.x * 4;
    if (c < d) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s = 0; s < n_splits; ++s) {
            const float ls = part_lse[s * stride + bh];
            if (ls == -INFINITY) continue;  // empty split: its partial rows were never written
            const float w = expf(ls - total);
            const float4 v = *reinterpret_cast<const float4*>(part_o + (s * stride + bh) * d + c);
            acc.x = fmaf(w, v.x, acc.x); acc.y = fmaf(w, v.y, acc.y);
            acc.z = fmaf(w, v.z, acc.z); acc.w = fmaf(w, v.w, acc.w);
        }
        uint2 w2;
        w2.x = pack_bf16x2(acc.x, acc.y);
        w2.y = pack_bf16x2(acc.z, acc.w);
        *reinterpret_cast<uint2*>(o + static_cast<size_t>(bh) * d + c) = w2;
    }
    if (threadIdx.x == 0) lse[static_cast<size_t>(h) * B + b] = total;
}

}  // namespace sdpa
