// Backward attention kernels for sm_100a.
//
// sdpa_bwd_preprocess_kernel : D_i = rowsum(dO * O) per (token, query head), fp32 [Hq, T]; clears
//                              the fp32 dQ accumulator.
// sdpa_bwd_kernel            : one CTA owns one 128-row key/value tile of one (sequence, kv head) and
//                              loops over the query heads of the group and over the 64-row query
//                              steps that can see it.  Scores are produced transposed (keys on TMEM
//                              lanes, queries on columns) so that P^T feeds dV += P^T dO straight from
//                              TMEM; dS^T goes through shared memory once and serves both
//                              dK += dS^T Q (as a K-major operand) and dQ = dS K (as an MN-major one).
//                              dK and dV stay in TMEM for the whole CTA; dQ steps are added into a
//                              head-major fp32 accumulator [Hq][T][D] with bulk reduce-adds.
// sdpa_bwd_dq_convert_kernel : fp32 dQ accumulator [Hq][T][D] * scale -> bf16 [T][Hq][D].
//
// Roles of sdpa_bwd_kernel (16 warps): warps 0-3 / 4-7 two compute groups (thread = key row, each
// group owns 32 of the 64 query columns of a step), warps 8-11 dQ reduction group, warps 12, 14, 15
// MMA issuers, warp 13 TMA producer.
// TMEM: S^T/P^T two 64-column buffers [0,128), dP^T then dQ^T two 64-column buffers [128,256),
// dV [256,256+D), dK [384,384+D).  Software pipeline: while the compute groups work on dS of step i and
// P of step i+1, the issuers run S^T(i+1), dV(i) / dK(i), dP^T(i+1) / dQ^T(i).  Buffer hazards:
// S^T(i+1) overwrites P^T(i-1) (same issuing thread as dV(i-1): in order); dP^T(i+1) overwrites
// dQ^T(i-1) (dq_empty: the reduction group has read it); dQ^T(i) overwrites dP^T(i) (ds_ready: the
// compute groups have read it); the dS^T buffer is reused after ds_free (both dK and dQ^T finished).
#pragma once
#include "ptx.cuh"
#include "layout.cuh"

namespace sdpa {

#ifdef SDPA_TRACE
__device__ long long g_trace[5 * 32 * 8];
#define SDPA_TR(role, it, k)                                                                   \
    do {                                                                                       \
        if (blockIdx.y == 0 && blockIdx.x == 4 * 8 && (it) >= 8 && (it) < 40)                       \
            g_trace[((role) * 32 + ((it) - 8)) * 8 + (k)] = clock64();                         \
    } while (0)
#else
#define SDPA_TR(role, it, k) do { } while (0)
#endif

struct BwdParams {
    const int32_t* cu_seqlens;
    const int32_t* cu_seqlens_k;  // key rows of sequence b in k / v / dk / dv (packed layout), or null: the query rows
    int Tk;                       // rows of k / v when cu_seqlens_k is given
    const float* lse;    // [Hq, T]
    const float* delta;  // [Hq, T]
    float* dq_acc;       // [Hq, T, D] fp32 (head-major; D = the kernel's padded head dimension)
    int* dq_turn;        // [Hq, T] turn counters of the deterministic mode (null otherwise), zeroed per call
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    int* status;
    int B, Hq, Hkv, T;
    int causal;
    int max_seqlen;
    int d;            // head dimension of the tensors (multiple of 8, <= D of the kernel; the rest is zero padding)
    TensorLayout lay;
    int group_chunk;  // (sequence, kv head) groups whose CTAs are launched interleaved
    float scale;
    float scale_log2;
};

template <int D>
struct BwdCfg {
    static constexpr int kThreads = 512;
    static constexpr int kTile = 128;
    static constexpr int kTileBytes = kTile * D * 2;
    static constexpr int kAtomBytes = kTile * 128;
    static constexpr int kStep = 64;                            // query rows per pipeline step
    static constexpr int kStepBytes = kStep * D * 2;            // one Q or dO step tile
    static constexpr int kStepAtomBytes = kStep * 128;          // one 64-column swizzle atom of a step tile
    static constexpr int kStageBytes = 2 * kStepBytes;          // Q step + dO step
    static constexpr int kQStages = 3;
    static constexpr int kSmemKV = 2 * kTileBytes;
    static constexpr int kSmemQdO = kQStages * kStageBytes;
    static constexpr int kSmemDS = 2 * 128 * 64 * 2;            // two dS^T buffers
    static constexpr int kSmemRows = kQStages * 2 * 64 * 4;     // lse / delta rows, one pair per Q/dO stage
    static constexpr int kSmemDQ = kStep * D * 4;               // fp32 staging of one dQ step for the bulk reduction
    static constexpr int kSmemBars = 256;
    // no alignment slack: the dynamic shared window is declared 1024-byte aligned and checked at run time
    static constexpr int kSmemBytes = kSmemKV + kSmemQdO + kSmemDS + kSmemDQ + kSmemRows + kSmemBars;
    static constexpr int kKSteps = D / 16;
};

enum BwdSite {
    kBSiteKvFull = 21, kBSiteQFull = 22, kBSiteQEmpty = 23, kBSiteSFull = 24, kBSiteDpFull = 25, kBSitePReady = 26,
    kBSiteDsReady = 27, kBSiteDsFree = 28, kBSiteDqFull = 29, kBSiteDqEmpty = 30, kBSiteDkvFull = 31, kBSiteDrain = 32, kBSiteTurn = 33
};

template <int D>
__global__ void __launch_bounds__(256)
sdpa_bwd_preprocess_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ dout,
                           float* __restrict__ delta, float* __restrict__ dq_acc, int* __restrict__ dq_turn, int T,
                           int Hq, int d, const TensorLayout lay) {
    constexpr int kLanesPerRow = D / 8;
    const long long gid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const long long row = gid / kLanesPerRow;  // row = global token * Hq + head
    const int part = static_cast<int>(gid % kLanesPerRow);
    const long long rows = static_cast<long long>(T) * Hq;
    float acc = 0.f;
    if (row < rows) {
        uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;  // padding columns d..D-1 contribute nothing
        if (part * 8 < d) {
            long long off = row * d + part * 8;  // packed [T, Hq, d]: rows are contiguous
            if (lay.dense) {
                const int gt = static_cast<int>(row / Hq), hh = static_cast<int>(row % Hq);
                off = (gt / lay.S) * lay.bs_q + static_cast<long long>(gt % lay.S) * lay.ts_q +
                      static_cast<long long>(hh) * lay.hs_q + part * 8;
            }
            a = *reinterpret_cast<const uint4*>(o + off);
            b = *reinterpret_cast<const uint4*>(dout + off);
        }
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w};
        const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            acc = fmaf(__uint_as_float(aw[i] << 16), __uint_as_float(bw[i] << 16), acc);
            acc = fmaf(__uint_as_float(aw[i] & 0xffff0000u), __uint_as_float(bw[i] & 0xffff0000u), acc);
        }
        float4* z = reinterpret_cast<float4*>(dq_acc + row * D + part * 8);
        z[0] = make_float4(0.f, 0.f, 0.f, 0.f);
        z[1] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int off = kLanesPerRow / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (row < rows && part == 0) {
        const long long tok = row / Hq;
        const int h = static_cast<int>(row % Hq);
        delta[static_cast<long long>(h) * T + tok] = acc;
        if (dq_turn != nullptr) dq_turn[static_cast<long long>(h) * T + tok] = 0;
    }
}

__global__ void __launch_bounds__(256)
sdpa_bwd_dq_convert_kernel(const float* __restrict__ dq_acc, __nv_bfloat16* __restrict__ dq, long long n8, float scale,
                           int T, int Hq, int D, int d, const TensorLayout lay) {
    // Blocks walk the tokens from the last one down: the rows the main kernel reduced into most recently are
    // still in the L2, the first ones are not; reading the hot rows first keeps them from being evicted by
    // this kernel's own traffic.
    const long long i = (static_cast<long long>(gridDim.x) - 1 - blockIdx.x) * blockDim.x + threadIdx.x;  // output group of 8
    if (i >= n8) return;
    const int d8 = d / 8;  // output rows have d columns, accumulator rows D (padded)
    const int part = static_cast<int>(i % d8);
    const long long th = i / d8;
    const int h = static_cast<int>(th % Hq);
    const long long t = th / Hq;
    const float* src = dq_acc + (static_cast<long long>(h) * T + t) * D + part * 8;
    const float4 a = reinterpret_cast<const float4*>(src)[0];
    const float4 b = reinterpret_cast<const float4*>(src)[1];
    uint4 w;
    w.x = pack_bf16x2(a.x * scale, a.y * scale);
    w.y = pack_bf16x2(a.z * scale, a.w * scale);
    w.z = pack_bf16x2(b.x * scale, b.y * scale);
    w.w = pack_bf16x2(b.z * scale, b.w * scale);
    long long off = i * 8;  // packed [T, Hq, d]: the output groups are contiguous
    if (lay.dense) {
        const int gt = static_cast<int>(t);
        off = (gt / lay.S) * lay.bs_q + static_cast<long long>(gt % lay.S) * lay.ts_q +
              static_cast<long long>(h) * lay.hs_q + part * 8;
    }
    *reinterpret_cast<uint4*>(dq + off) = w;
}

template <int D>
__global__ void __launch_bounds__(512, 1)
sdpa_bwd_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do,
                const BwdParams p) {
    using Cfg = BwdCfg<D>;
    constexpr int NS = Cfg::kQStages;
    // Launch order: the (sequence, kv head) groups are taken in chunks of p.group_chunk; inside a chunk the
    // CTAs go key tile by key tile (under a causal mask the low key tiles see the most queries, so the heavy
    // CTAs start first), chunk after chunk.  CTAs that run at the same time therefore belong to few groups
    // and sweep the same query heads at about the same time, which keeps the part of the fp32 dQ accumulator
    // being reduced into inside the L2; one chunk for everything would spread a wave over all groups and
    // every accumulator line would travel to DRAM and back once per wave.
    const int bg = static_cast<int>(blockIdx.y) * p.group_chunk + static_cast<int>(blockIdx.x) % p.group_chunk;
    if (bg >= p.B * p.Hkv) return;
    const int b = bg / p.Hkv, g = bg % p.Hkv;
    const int G = p.Hq / p.Hkv;
    SeqPos sp;
    if (!locate_sequence(p.lay, p.cu_seqlens, b, p.T, p.max_seqlen, sp)) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0, kStatusBadCuSeqlens);
        return;
    }
    const int r0 = sp.tok0;  // token coordinate of the sequence's first row in the tensors
    const int L = sp.L;
    // causal: low key tiles see the most query tiles -> launch them first
    const int n_tiles_grid = static_cast<int>(gridDim.x) / p.group_chunk;
    const int jt_raw = static_cast<int>(blockIdx.x) / p.group_chunk;
    // The deterministic mode launches the high (light) key tiles first, so that a tile only ever waits for
    // tiles launched before it (see the turn counters in the reduction group).
    const int jt = (p.causal && p.dq_turn == nullptr) ? jt_raw : n_tiles_grid - 1 - jt_raw;
    const int kv0 = jt * 128;
    // Keys of the sequence: the rows of its queries, or a row range of their own with Lk keys for L queries;
    // a causal query i then sees keys 0 .. i + off, off = Lk - L (the last query sees the last key).
    int rk0 = r0, Lk = L;
    if (p.cu_seqlens_k != nullptr) {
        rk0 = p.cu_seqlens_k[b];
        const int rk1 = p.cu_seqlens_k[b + 1];
        Lk = rk1 - rk0;
        if (rk0 < 0 || rk1 > p.Tk || Lk < 0 || (L > 0 && (Lk < 1 || (p.causal && Lk < L)))) {
            if (threadIdx.x == 0) atomicCAS(p.status, 0, kStatusBadCuSeqlens);
            return;
        }
    }
    const int off = Lk - L;
    if (kv0 >= Lk) return;
    if (L == 0) {
        // keys without any query: their gradients are zero (only possible with separate key lengths)
        const int rows = min(128, Lk - kv0), d8 = p.d >> 3;
        for (int i = threadIdx.x; i < rows * d8; i += blockDim.x) {
            const long long o8 = static_cast<long long>(rk0 + kv0 + i / d8) * p.lay.ts_kv +
                                 static_cast<long long>(g) * p.lay.hs_kv + (i % d8) * 8;
            *reinterpret_cast<uint4*>(p.dk + o8) = make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(p.dv + o8) = make_uint4(0u, 0u, 0u, 0u);
        }
        return;
    }
    const int n_qs = (L + 63) >> 6;            // 64-row query steps in the sequence
    const int i_start = p.causal ? max(0, kv0 - off) >> 6 : 0;  // first query step that sees this key tile
    const int per_head = n_qs - i_start;
    const int n_it = G * per_head;
    const bool det = p.dq_turn != nullptr;
    const int nt_seq = (Lk + 127) >> 7;  // key tiles of this sequence
    auto step_of = [&](int it) { return i_start + it % per_head; };

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = smem_raw;
    if ((smem_u32(smem) & 1023u) != 0u) {  // swizzled tiles need 1024-byte alignment
        if (threadIdx.x == 0) atomicCAS(p.status, 0, kStatusInternal);
        return;
    }
    uint8_t* sK = smem;
    uint8_t* sV = smem + Cfg::kTileBytes;
    uint8_t* sQdO = smem + Cfg::kSmemKV;  // stage s: Q step at s*kStageBytes, dO step right after it
    uint8_t* sDS = sQdO + Cfg::kSmemQdO;  // two buffers of [128 keys][64 queries] bf16, swizzled
    float* sDQ = reinterpret_cast<float*>(sDS + Cfg::kSmemDS);    // [64 queries][D] fp32
    float* sRows = reinterpret_cast<float*>(sDS + Cfg::kSmemDS + Cfg::kSmemDQ);  // [NS stages][lse2 | delta][64]
    uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(sRows) + Cfg::kSmemRows);
    uint64_t* kv_full = bars;             // 1
    uint64_t* q_full = bars + 1;          // NS
    uint64_t* q_empty = q_full + NS;      // NS
    uint64_t* s_full = q_empty + NS;      // 2
    uint64_t* dp_full = s_full + 2;       // 2
    uint64_t* p_ready = dp_full + 2;      // 2
    uint64_t* ds_ready = p_ready + 2;     // 2
    uint64_t* ds_free = ds_ready + 2;     // 2
    uint64_t* dq_full = ds_free + 2;      // 2
    uint64_t* dq_empty = dq_full + 2;     // 2
    uint64_t* dkv_full = dq_empty + 2;    // 1
    uint64_t* drain = dkv_full + 1;       // 3
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 3);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const WaitCtl ctl{p.status, abort_flag};

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(kv_full, 1);
        for (int i = 0; i < NS; ++i) {
            mbar_init(&q_full[i], 33);  // TMA transaction arrival + 32 lanes that staged the lse / D_i rows
            mbar_init(&q_empty[i], 3);  // one commit per MMA-issuing warp
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s_full[i], 1);
            mbar_init(&dp_full[i], 1);
            mbar_init(&p_ready[i], 128);
            mbar_init(&ds_ready[i], 128);
            mbar_init(&ds_free[i], 2);  // dK issuer and dQ^T issuer
            mbar_init(&dq_full[i], 1);
            mbar_init(&dq_empty[i], 128);
        }
        mbar_init(dkv_full, 2);
        for (int i = 0; i < 3; ++i) mbar_init(&drain[i], 1);
        fence_mbar_init();
    }
    if (warp == 12) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    if (warp == 13 && elect_one()) {
        prefetch_tmap(&map_q);
        prefetch_tmap(&map_k);
        prefetch_tmap(&map_v);
        prefetch_tmap(&map_do);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    // TMEM columns: S^T/P^T two buffers of 64, dP^T/dQ^T two buffers of 64, dV, dK
    constexpr uint32_t kColS = 0, kColDP = 128, kColDV = 256, kColDK = 384;

    // Register re-balancing: one setmaxnreg instruction per warpgroup, executed by all of its warps.
    if (warp < 8) setmaxnreg_inc<168>();
    else setmaxnreg_dec<88>();

    if (warp < 8) {
        // ------------------------------------------------------------ compute groups (ping-pong over steps)
        // Group w owns the steps of parity w and the TMEM / dS buffers of index w, so one group's
        // exponentials overlap the other group's dS and the MMAs of both.
        const int wg = warp >> 2;
        const int r = tid & 127;           // key row inside the tile
        const int key = kv0 + r;           // key index inside the sequence
        const bool key_ok = key < Lk;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_base + kColS + wg * 64;
        const uint32_t tDP = tmem + lane_base + kColDP + wg * 64;
        uint8_t* ds_buf = sDS + wg * 16384;
        bool ok = true;
        uint32_t stage = wg % NS, sphase = 0;
        for (int s = wg; s < n_it && ok; s += 2) {
            const uint32_t ph = (s >> 1) & 1;
            const int q0 = step_of(s) * 64;
            const bool need_mask = (p.causal && q0 + off < kv0 + 128) || (kv0 + 128 > Lk);
            // rows (lse * log2e, D_i) of this step were staged by the producer warp together with Q / dO
            if (r == 0) SDPA_TR(0, s, 0);
            ok = mbar_wait_warp(&q_full[stage], sphase, ctl, kBSiteQFull);
            if (!ok) break;
            const float4* lse4 = reinterpret_cast<const float4*>(sRows + stage * 128);
            const float4* dl4 = reinterpret_cast<const float4*>(sRows + stage * 128 + 64);
            // A(s): P^T = exp2(S^T * scale_log2 - lse2) with masks; bf16 P^T overwrites the S^T columns
            ok = mbar_wait_warp(&s_full[wg], ph, ctl, kBSiteSFull);
            if (!ok) break;
            if (r == 0) SDPA_TR(0, s, 1);
            tc_fence_after();
            float pr[64];
            uint32_t sr_all[2][32];  // both halves of the step's scores are requested before the first wait
            tmem_ld_x32(tS, sr_all[0]);
            tmem_ld_x32(tS + 32, sr_all[1]);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const uint32_t (&sr)[32] = sr_all[c];
#pragma unroll
                for (int i4 = 0; i4 < 8; ++i4) {
                    const float4 l4 = lse4[c * 8 + i4];
                    const float lv[4] = {l4.x, l4.y, l4.z, l4.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int i = i4 * 4 + e;
                        pr[c * 32 + i] = fast_exp2(fmaf(__uint_as_float(sr[i]), p.scale_log2, -lv[e]));
                    }
                }
                if (need_mask) {  // diagonal and tail steps only: kept out of the common path
                    const int q_lim = key - off;  // under a causal mask this key is seen by queries >= q_lim
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (!key_ok || (p.causal && q0 + c * 32 + i < q_lim)) pr[c * 32 + i] = 0.f;
                }
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) pk[i] = pack_bf16x2(pr[c * 32 + 2 * i], pr[c * 32 + 2 * i + 1]);
                tmem_st_x16(tS + c * 16, pk);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&p_ready[wg]);
            if (r == 0) SDPA_TR(0, s, 2);
            // B(s): dS^T = P^T * (dP^T - D_i) -> bf16 -> swizzled shared memory
            ok = mbar_wait_warp(&dp_full[wg], ph, ctl, kBSiteDpFull);
            if (!ok) break;
            if (r == 0) SDPA_TR(0, s, 3);
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t dr[32];
                tmem_ld_x32(tDP + c * 32, dr);
                tmem_wait_ld();
#pragma unroll
                for (int i4 = 0; i4 < 8; ++i4) {
                    const float4 d4 = dl4[c * 8 + i4];
                    pr[c * 32 + i4 * 4 + 0] *= (__uint_as_float(dr[i4 * 4 + 0]) - d4.x);
                    pr[c * 32 + i4 * 4 + 1] *= (__uint_as_float(dr[i4 * 4 + 1]) - d4.y);
                    pr[c * 32 + i4 * 4 + 2] *= (__uint_as_float(dr[i4 * 4 + 2]) - d4.z);
                    pr[c * 32 + i4 * 4 + 3] *= (__uint_as_float(dr[i4 * 4 + 3]) - d4.w);
                }
            }
            if (s >= 2) {
                ok = mbar_wait_warp(&ds_free[wg], ph ^ 1, ctl, kBSiteDsFree);
                if (!ok) break;
            }
            if (r == 0) SDPA_TR(0, s, 4);
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
                uint4 w;
                w.x = pack_bf16x2(pr[ch * 8 + 0], pr[ch * 8 + 1]);
                w.y = pack_bf16x2(pr[ch * 8 + 2], pr[ch * 8 + 3]);
                w.z = pack_bf16x2(pr[ch * 8 + 4], pr[ch * 8 + 5]);
                w.w = pack_bf16x2(pr[ch * 8 + 6], pr[ch * 8 + 7]);
                *reinterpret_cast<uint4*>(ds_buf + sw128_offset(r, ch)) = w;
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(&ds_ready[wg]);
            if (r == 0) SDPA_TR(0, s, 5);
            stage += 2;
            if (stage >= NS) { stage -= NS; sphase ^= 1; }
        }
        if (ok) ok = mbar_wait_warp(dkv_full, 0, ctl, kBSiteDkvFull);
        if (ok) {
            tc_fence_after();
            // group 0 writes dV, group 1 writes dK (scaled)
            const uint32_t tAcc = tmem + lane_base + (wg == 0 ? kColDV : kColDK);
            const float mul = wg == 0 ? 1.0f : p.scale;
            __nv_bfloat16* out = wg == 0 ? p.dv : p.dk;
            // The rows leave through shared memory that no MMA reads any more once dkv_full has completed: the
            // V tile (group 0; its last reader dP^T finished before the last dS) and the first Q/dO stage
            // (group 1; the K tile may still feed the last dQ^T).  Each thread writes its bf16 row there
            // (16-byte chunks XOR-swizzled by row), then each warp copies its own 32 rows out with full-line
            // stores instead of 32 different lines per store.
            constexpr int kChunks = D / 8;
            constexpr int kRowsPerPass = 32 / kChunks;
            uint8_t* out_stage = wg == 0 ? sV : sQdO;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t a[32];
                tmem_ld_x32(tAcc + c * 32, a);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 w;
                    w.x = pack_bf16x2(__uint_as_float(a[8 * i + 0]) * mul, __uint_as_float(a[8 * i + 1]) * mul);
                    w.y = pack_bf16x2(__uint_as_float(a[8 * i + 2]) * mul, __uint_as_float(a[8 * i + 3]) * mul);
                    w.z = pack_bf16x2(__uint_as_float(a[8 * i + 4]) * mul, __uint_as_float(a[8 * i + 5]) * mul);
                    w.w = pack_bf16x2(__uint_as_float(a[8 * i + 6]) * mul, __uint_as_float(a[8 * i + 7]) * mul);
                    const int k = c * 4 + i;
                    *reinterpret_cast<uint4*>(out_stage + r * (D * 2) + ((k ^ (r & 7)) << 4)) = w;
                }
            }
            __syncwarp();
            {
                const int lane = tid & 31;
                const int k = lane % kChunks;
                const int rows_left = Lk - kv0;  // keys of this tile inside the sequence
#pragma unroll
                for (int pass = 0; pass < 32 / kRowsPerPass; ++pass) {
                    const int rr = (warp & 3) * 32 + pass * kRowsPerPass + lane / kChunks;
                    if (rr < rows_left && k * 8 < p.d) {
                        const uint4 w = *reinterpret_cast<const uint4*>(out_stage + rr * (D * 2) + ((k ^ (rr & 7)) << 4));
                        __nv_bfloat16* dst = out + sp.bidx * p.lay.bs_kv +
                                             static_cast<long long>(rk0 + kv0 + rr) * p.lay.ts_kv +
                                             static_cast<long long>(g) * p.lay.hs_kv;
                        *reinterpret_cast<uint4*>(dst + k * 8) = w;
                    }
                }
            }
        }
    } else if (warp < 12) {
        // ------------------------------------------------------------ dQ reduction group
        // dQ^T step: TMEM lane = d, columns = 64 queries.  The step is transposed into shared memory as
        // [query][d] fp32 (one warp store = 128 contiguous bytes) and added to the head-major fp32
        // accumulator [Hq][T][D] with ONE bulk reduce-add of up to 64*D*4 contiguous bytes.
        const int x = tid & 127;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        bool ok = true;
        // Deterministic mode: the key tiles that see a query step add into it from the highest tile index
        // down.  That is the order in which they reach the step anyway (tile j starts its sweep at step 2j
        // under a causal mask), and the tiles waited for were launched earlier.  The counter of a step holds
        // how many tiles have added.  Thread 32 waits for this tile's rank while the group stages the step;
        // thread 0 adds and passes the turn on two steps later, when `cp.async.bulk.wait_group 2` says that
        // the adds have been performed: their latency (L2 reduce throughput plus a round trip) is longer
        // than one step.  A wait that gives up raises the CTA's abort flag; the adds are then skipped.
        // turn counter of iteration i and this tile's rank on it (pure functions of i: nothing is carried
        // from step to step in registers)
        auto turn_of = [&](int i, int& rank) -> int* {
            const int hh = g * G + i / per_head;
            const int qq0 = step_of(i) * 64;
            const int j_last = p.causal ? min(nt_seq - 1, (qq0 + 63 + off) >> 7) : nt_seq - 1;  // highest tile on the step
            rank = j_last - jt;
            return p.dq_turn + static_cast<size_t>(hh) * p.T + sp.gt0 + qq0;
        };
        for (int it = 0; it < n_it && ok; ++it) {
            const int h = g * G + it / per_head;
            const int q0 = step_of(it) * 64;
            if (x == 0) SDPA_TR(4, it, 0);
            ok = mbar_wait_warp(&dq_full[it & 1], (it >> 1) & 1, ctl, kBSiteDqFull);
            if (!ok) break;
            if (x == 0) SDPA_TR(4, it, 1);
            tc_fence_after();
            const uint32_t tDQ = tmem + lane_base + kColDP + (it & 1) * 64;
            uint32_t a0[32], a1[32];
            tmem_ld_x32(tDQ, a0);
            tmem_ld_x32(tDQ + 32, a1);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(&dq_empty[it & 1]);
            if (x == 0) SDPA_TR(4, it, 2);
            if (det) {
                if (x == 32) {
                    int rank;
                    int* turn = turn_of(it, rank);
                    wait_turn(turn, rank, ctl, kBSiteTurn);  // sets the abort flag on failure
                }
                if (x == 0 && it >= 2) {
                    bulk_wait<2>();  // all but the previous step's two groups: the adds of two steps ago are done
                    int rank;
                    int* turn = turn_of(it - 2, rank);
                    if (!*ctl.abort) release_turn(turn, rank + 1);
                }
            }
            // Two halves of 32 query rows, each its own bulk group: the rows of one half are rewritten
            // while the bulk engine is still reading the other half of the previous step.
            const int nq = min(64, L - q0);
            float* dst = p.dq_acc + (static_cast<size_t>(h) * p.T + sp.gt0 + q0) * D;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                if (x == 0) bulk_wait_read<1>();  // the group that last read this half has finished reading
                named_bar_sync(2, 128);
                if (x < D) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        sDQ[(hf * 32 + i) * D + x] = __uint_as_float(hf == 0 ? a0[i] : a1[i]);
                }
                fence_proxy_async_smem();
                named_bar_sync(2, 128);
                if (x == 0) {
                    const int rows = min(32, nq - hf * 32);
                    if (rows > 0 && !(det && *ctl.abort))
                        bulk_reduce_add_f32(dst + hf * 32 * D, sDQ + hf * 32 * D, static_cast<uint32_t>(rows) * D * 4u);
                    bulk_commit();  // committed even when empty, so the group count per step is fixed
                }
                if (x == 0 && hf == 0) SDPA_TR(4, it, 3);
            }
            if (x == 0) SDPA_TR(4, it, 4);
            if (x == 0) SDPA_TR(4, it, 5);
        }
        if (x == 0) {
            bulk_wait<0>();
            if (det && ok && !*ctl.abort) {
                for (int i = max(0, n_it - 2); i < n_it; ++i) {
                    int rank;
                    int* turn = turn_of(i, rank);
                    release_turn(turn, rank + 1);
                }
            }
        }
    } else if (warp == 13) {
        // ------------------------------------------------------------ producer warp (all 32 lanes)
        // Lane 0 issues the TMA loads; every lane stages two (lse * log2e, D_i) pairs of the step's 64
        // query rows in shared memory.  q_full collects the TMA bytes and the 32 lane arrivals.
        const int lane = tid & 31;
        if (lane == 0) {
            mbar_arrive_expect_tx(kv_full, 2 * Cfg::kTileBytes);
#pragma unroll
            for (int a = 0; a < D / 64; ++a) {
                SDPA_TMA_LOAD_ROWS(sK + a * Cfg::kAtomBytes, &map_k, kv_full, a * 64, rk0 + kv0, g, sp.bidx, p.lay.dense);
                SDPA_TMA_LOAD_ROWS(sV + a * Cfg::kAtomBytes, &map_v, kv_full, a * 64, rk0 + kv0, g, sp.bidx, p.lay.dense);
            }
        }
        bool ok = true;
        int it = 0;
        uint32_t st = 0, ph = 0;
        for (; it < n_it && ok; ++it) {
            ok = mbar_wait_warp(&q_empty[st], ph ^ 1, ctl, kBSiteQEmpty);
            if (!ok) break;
            const int h = g * G + it / per_head;
            const int q0 = step_of(it) * 64;
            if (lane == 0) {
                uint8_t* dst = sQdO + st * Cfg::kStageBytes;
                mbar_arrive_expect_tx(&q_full[st], Cfg::kStageBytes);
#pragma unroll
                for (int a = 0; a < D / 64; ++a) {
                    SDPA_TMA_LOAD_ROWS(dst + a * Cfg::kStepAtomBytes, &map_q, &q_full[st], a * 64, r0 + q0, h, sp.bidx, p.lay.dense);
                    SDPA_TMA_LOAD_ROWS(dst + Cfg::kStepBytes + a * Cfg::kStepAtomBytes, &map_do, &q_full[st], a * 64, r0 + q0,
                                h, sp.bidx, p.lay.dense);
                }
            }
            float* rows = sRows + st * 128;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int qi = lane * 2 + e;
                float lv = INFINITY, dv = 0.f;  // rows past the sequence end: P = exp2(-inf) = 0
                if (q0 + qi < L) {
                    lv = p.lse[sp.bidx * p.lay.lse_bs + static_cast<long long>(h) * p.lay.lse_hs + r0 + q0 + qi] *
                         1.4426950408889634f;
                    dv = p.delta[static_cast<size_t>(h) * p.T + sp.gt0 + q0 + qi];
                }
                rows[qi] = lv;
                rows[64 + qi] = dv;
            }
            mbar_arrive(&q_full[st]);
            if (++st == NS) { st = 0; ph ^= 1; }
        }
        if (!ok && lane == 0) {
            mbar_wait(kv_full, 0, ctl, kBSiteDrain);
            for (int back = 1; back <= NS && back <= it; ++back) {
                const int i2 = it - back;
                mbar_wait(&q_full[i2 % NS], (i2 / NS) & 1, ctl, kBSiteDrain);
            }
        }
    } else {
        // ------------------------------------------------------------ MMA issuers (warps 12, 14, 15)
        // The issuing thread's own instruction stream bounds its MMA rate, so the MMAs of a step are
        // spread over three warps:  warp 12: dV(i), S^T(i+2);  warp 14: dK(i);
        // warp 15: dQ^T(i), then (after the reduction group drained it) dP^T(i+2) into the same columns.
        if (elect_one()) {
            constexpr uint32_t idesc_s = make_idesc_bf16(128, 64, false, false);   // S^T, dP^T: keys x 64 queries
            constexpr uint32_t idesc_acc = make_idesc_bf16(128, D, false, true);   // dV, dK: keys x d
            constexpr uint32_t idesc_dq = make_idesc_bf16(128, 64, true, true);    // dQ^T: d x 64 queries
            constexpr uint32_t kLboK = (D == 128) ? Cfg::kAtomBytes : 0;           // D=64: rows 64..127 repeat, unused
            constexpr uint64_t kStageStep = Cfg::kStageBytes >> 4;
            constexpr uint64_t kDsStep = 16384 >> 4;
            auto kmaj = [](int kk, int atom_bytes) -> uint64_t {
                return static_cast<uint64_t>(((kk >> 2) * atom_bytes + (kk & 3) * 32) >> 4);
            };
            bool ok = mbar_wait(kv_full, 0, ctl, kBSiteKvFull);
            if (warp == 12) {
                const uint64_t k_desc = smem_desc_sw128(smem_u32(sK), 0, 1024);
                const uint64_t q_desc = smem_desc_sw128(smem_u32(sQdO), 0, 1024);                               // K-major B
                const uint64_t do_mn_desc = smem_desc_sw128(smem_u32(sQdO) + Cfg::kStepBytes, Cfg::kStepAtomBytes, 1024);  // MN-major B
                auto issue_s = [&](uint32_t buf, uint32_t stage) {  // S^T = K Q^T into S buffer `buf`
                    const uint64_t qd = q_desc + stage * kStageStep;
                    const uint32_t d = tmem + kColS + buf * 64;
#pragma unroll
                    for (int kk = 0; kk < Cfg::kKSteps; ++kk)
                        umma_ss(d, k_desc + kmaj(kk, Cfg::kAtomBytes), qd + kmaj(kk, Cfg::kStepAtomBytes), idesc_s, kk > 0);
                };
                // prologue: S^T(0), S^T(1)
                for (int s = 0; s < 2 && s < n_it && ok; ++s) {
                    ok = mbar_wait(&q_full[s % NS], 0, ctl, kBSiteQFull);
                    if (!ok) break;
                    tc_fence_after();
                    issue_s(s, s % NS);
                    umma_commit(&s_full[s]);
                }
                uint32_t stage = 0;                        // stage of step it
                uint32_t stage2 = 2 % NS, phase2 = (2 >= NS) ? 1u : 0u;  // stage / phase of step it+2
                for (int it = 0; it < n_it && ok; ++it) {
                    const uint32_t buf = it & 1, ph = (it >> 1) & 1;
                    SDPA_TR(1, it, 0);
                    // dV += P^T dO   (P^T from TMEM; the 64 queries of the step are the contraction index)
                    ok = mbar_wait(&p_ready[buf], ph, ctl, kBSitePReady);
                    if (!ok) break;
                    SDPA_TR(1, it, 1);
                    tc_fence_after();
                    {
                        const uint64_t dod = do_mn_desc + stage * kStageStep;
                        const uint32_t a = tmem + kColS + buf * 64;
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            umma_ts(tmem + kColDV, a + kk * 8, dod + static_cast<uint64_t>(kk * (2048 >> 4)), idesc_acc,
                                    (it > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(&q_empty[stage]);
                    SDPA_TR(1, it, 2);
                    if (it + 2 < n_it) {  // S^T(it+2) overwrites P^T(it): same thread, issued in order after dV(it)
                        ok = mbar_wait(&q_full[stage2], phase2, ctl, kBSiteQFull);
                        if (!ok) break;
                        SDPA_TR(1, it, 3);
                        tc_fence_after();
                        issue_s(buf, stage2);
                        umma_commit(&s_full[buf]);
                        SDPA_TR(1, it, 4);
                    }
                    if (++stage == NS) stage = 0;
                    if (++stage2 == NS) { stage2 = 0; phase2 ^= 1; }
                }
                if (ok) umma_commit(dkv_full);
            } else if (warp == 14) {
                const uint64_t q_mn_desc = smem_desc_sw128(smem_u32(sQdO), Cfg::kStepAtomBytes, 1024);           // MN-major B
                const uint64_t ds_desc = smem_desc_sw128(smem_u32(sDS), 0, 1024);                                // K-major A
                uint32_t stage = 0;
                for (int it = 0; it < n_it && ok; ++it) {
                    const uint32_t buf = it & 1, ph = (it >> 1) & 1;
                    // dK += dS^T Q
                    SDPA_TR(2, it, 0);
                    ok = mbar_wait(&ds_ready[buf], ph, ctl, kBSiteDsReady);
                    if (!ok) break;
                    SDPA_TR(2, it, 1);
                    tc_fence_after();
                    const uint64_t dsd = ds_desc + buf * kDsStep;
                    const uint64_t qd = q_mn_desc + stage * kStageStep;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_ss(tmem + kColDK, dsd + static_cast<uint64_t>(kk * 2), qd + static_cast<uint64_t>(kk * (2048 >> 4)),
                                idesc_acc, (it > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(&ds_free[buf]);
                    umma_commit(&q_empty[stage]);
                    SDPA_TR(2, it, 2);
                    if (++stage == NS) stage = 0;
                }
                if (ok) umma_commit(dkv_full);
            } else {
                const uint64_t kt_desc = smem_desc_sw128(smem_u32(sK), kLboK, 1024);                             // MN-major A
                const uint64_t ds_mn_desc = smem_desc_sw128(smem_u32(sDS), 0, 1024);                             // MN-major B
                const uint64_t v_desc = smem_desc_sw128(smem_u32(sV), 0, 1024);
                const uint64_t do_desc = smem_desc_sw128(smem_u32(sQdO) + Cfg::kStepBytes, 0, 1024);            // K-major B
                auto issue_dp = [&](uint32_t buf, uint32_t stage) {  // dP^T = V dO^T into dP buffer `buf`
                    const uint64_t dd = do_desc + stage * kStageStep;
                    const uint32_t d = tmem + kColDP + buf * 64;
#pragma unroll
                    for (int kk = 0; kk < Cfg::kKSteps; ++kk)
                        umma_ss(d, v_desc + kmaj(kk, Cfg::kAtomBytes), dd + kmaj(kk, Cfg::kStepAtomBytes), idesc_s, kk > 0);
                };
                // Event loop: issue whichever of dP^T(np) / dQ^T(nq) has its inputs ready, so that waiting
                // for the reduction group to drain one buffer never delays the other buffer's dQ^T.
                int nq = 0, np = 0;
                uint32_t stage_p = 0, phase_p = 0;  // Q/dO stage and phase of step np
                long long t_idle = 0;
                bool idle = false;
                while (ok && (nq < n_it || np < n_it)) {
                    bool did = false;
                    if (np < n_it && np < nq + 2) {
                        // dP^T(np) reuses the columns of dQ^T(np-2): wait until the reduction group has read it
                        if (mbar_test_wait(&q_full[stage_p], phase_p) &&
                            (np < 2 || mbar_test_wait(&dq_empty[np & 1], ((np >> 1) - 1) & 1))) {
                            SDPA_TR(3, np, 3);
                            tc_fence_after();
                            issue_dp(np & 1, stage_p);
                            umma_commit(&dp_full[np & 1]);
                            umma_commit(&q_empty[stage_p]);
                            SDPA_TR(3, np, 4);
                            ++np;
                            if (++stage_p == NS) { stage_p = 0; phase_p ^= 1; }
                            did = true;
                        }
                    }
                    if (!did && nq < n_it && mbar_test_wait(&ds_ready[nq & 1], (nq >> 1) & 1)) {
                        SDPA_TR(3, nq, 1);
                        tc_fence_after();
                        // dQ^T = K^T dS^T (overwrites the dP^T buffer of this step)
                        const uint64_t dsd = ds_mn_desc + (nq & 1) * kDsStep;
                        const uint32_t d = tmem + kColDP + (nq & 1) * 64;
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)
                            umma_ss(d, kt_desc + static_cast<uint64_t>(kk * (2048 >> 4)), dsd + static_cast<uint64_t>(kk * (2048 >> 4)),
                                    idesc_dq, kk > 0);
                        umma_commit(&dq_full[nq & 1]);
                        umma_commit(&ds_free[nq & 1]);
                        SDPA_TR(3, nq, 2);
                        ++nq;
                        did = true;
                    }
                    if (did) {
                        idle = false;
                    } else if (!idle) {
                        idle = true;
                        t_idle = clock64();
                    } else if (*ctl.abort) {
                        ok = false;
                    } else if (clock64() - t_idle > ctl.limit) {
                        *ctl.abort = 1;
                        atomicCAS(ctl.g_status, 0, (kBSiteDqEmpty << 8) | kStatusTimeout);
                        ok = false;
                    }
                }
            }
            if (!ok) {
                uint64_t* my_drain = &drain[warp == 12 ? 0 : (warp == 14 ? 1 : 2)];
                umma_commit(my_drain);
                mbar_wait(my_drain, 0, ctl, kBSiteDrain);
            }
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 12) tmem_dealloc(tmem, 512);
}

}  // namespace sdpa
