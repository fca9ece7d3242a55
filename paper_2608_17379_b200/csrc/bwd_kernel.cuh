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

namespace sdpa {

#ifdef SDPA_TRACE
__device__ long long g_trace[5 * 32 * 8];
#define SDPA_TR(role, it, k)                                                                   \
    do {                                                                                       \
        if (blockIdx.x == 0 && blockIdx.y == 4 && (it) >= 8 && (it) < 40)                       \
            g_trace[((role) * 32 + ((it) - 8)) * 8 + (k)] = clock64();                         \
    } while (0)
#else
#define SDPA_TR(role, it, k) do { } while (0)
#endif

struct BwdParams {
    const int32_t* cu_seqlens;
    const float* lse;    // [Hq, T]
    const float* delta;  // [Hq, T]
    float* dq_acc;       // [Hq, T, D] fp32 (head-major)
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    int* status;
    int B, Hq, Hkv, T;
    int causal;
    int max_seqlen;
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
    static constexpr int kSmemRows = 2 * 2 * 64 * 4;            // lse / delta rows, double buffered
    static constexpr int kSmemDQ = kStep * D * 4;               // fp32 staging of one dQ step for the bulk reduction
    static constexpr int kSmemBars = 256;
    // no alignment slack: the dynamic shared window is declared 1024-byte aligned and checked at run time
    static constexpr int kSmemBytes = kSmemKV + kSmemQdO + kSmemDS + kSmemDQ + kSmemRows + kSmemBars;
    static constexpr int kKSteps = D / 16;
};

enum BwdSite {
    kBSiteKvFull = 21, kBSiteQFull = 22, kBSiteQEmpty = 23, kBSiteSFull = 24, kBSiteDpFull = 25, kBSitePReady = 26,
    kBSiteDsReady = 27, kBSiteDsFree = 28, kBSiteDqFull = 29, kBSiteDqEmpty = 30, kBSiteDkvFull = 31, kBSiteDrain = 32
};

template <int D>
__global__ void __launch_bounds__(256)
sdpa_bwd_preprocess_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ dout,
                           float* __restrict__ delta, float* __restrict__ dq_acc, int T, int Hq) {
    constexpr int kLanesPerRow = D / 8;
    const long long gid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const long long row = gid / kLanesPerRow;  // row = token * Hq + head
    const int part = static_cast<int>(gid % kLanesPerRow);
    const long long rows = static_cast<long long>(T) * Hq;
    float acc = 0.f;
    if (row < rows) {
        const uint4 a = *reinterpret_cast<const uint4*>(o + row * D + part * 8);
        const uint4 b = *reinterpret_cast<const uint4*>(dout + row * D + part * 8);
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
    }
}

__global__ void __launch_bounds__(256)
sdpa_bwd_dq_convert_kernel(const float* __restrict__ dq_acc, __nv_bfloat16* __restrict__ dq, long long n8, float scale,
                           int T, int Hq, int D) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;  // output group of 8
    if (i >= n8) return;
    const int d8 = D / 8;
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
    reinterpret_cast<uint4*>(dq)[i] = w;
}

template <int D>
__global__ void __launch_bounds__(512, 1)
sdpa_bwd_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do,
                const BwdParams p) {
    using Cfg = BwdCfg<D>;
    constexpr int NS = Cfg::kQStages;
    const int bg = blockIdx.x;
    const int b = bg / p.Hkv, g = bg % p.Hkv;
    const int G = p.Hq / p.Hkv;
    const int r0 = p.cu_seqlens[b];
    const int r1 = p.cu_seqlens[b + 1];
    const int L = r1 - r0;
    if (L < 0 || r0 < 0 || r1 > p.T || L > p.max_seqlen) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0, kStatusBadCuSeqlens);
        return;
    }
    // causal: low key tiles see the most query tiles -> launch them first
    const int jt = p.causal ? static_cast<int>(blockIdx.y) : static_cast<int>(gridDim.y) - 1 - static_cast<int>(blockIdx.y);
    const int kv0 = jt * 128;
    if (kv0 >= L) return;
    const int n_qs = (L + 63) >> 6;            // 64-row query steps in the sequence
    const int i_start = p.causal ? 2 * jt : 0;  // first query step that sees this key tile
    const int per_head = n_qs - i_start;
    const int n_it = G * per_head;

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
    float* sRows = reinterpret_cast<float*>(sDS + Cfg::kSmemDS + Cfg::kSmemDQ);  // [2 buffers][lse2 | delta][64]
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
            mbar_init(&q_full[i], 1);
            mbar_init(&q_empty[i], 2);  // released by the S^T/dV issuer and by the dP^T/dK issuer
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s_full[i], 1);
            mbar_init(&dp_full[i], 1);
            mbar_init(&p_ready[i], 256);
            mbar_init(&ds_ready[i], 256);
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

    if (warp < 8) {
        // ------------------------------------------------------------ compute groups
        const int wg = warp >> 2;          // owns query columns [32*wg, 32*wg + 32) of every step
        const int r = tid & 127;           // key row inside the tile
        const int key = kv0 + r;           // key index inside the sequence
        const bool key_ok = key < L;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const int row_which = tid >> 6, row_qi = tid & 63;  // threads 0..127 stage lse / delta rows
        auto load_row = [&](int s) -> float {
            float val = row_which == 0 ? INFINITY : 0.f;
            if (tid < 128 && s < n_it) {
                const int h = g * G + s / per_head;
                const int qrow = (i_start + s % per_head) * 64 + row_qi;
                if (qrow < L) {
                    const size_t idx = static_cast<size_t>(h) * p.T + r0 + qrow;
                    val = row_which == 0 ? p.lse[idx] * 1.4426950408889634f : p.delta[idx];
                }
            }
            return val;
        };
        float pr[32];
        bool ok = true;
        // A(s): P^T = exp2(S^T * scale_log2 - lse2) with masks; bf16 P^T overwrites the S^T columns
        auto stage_a = [&](int s) -> bool {
            if (tid == 0) SDPA_TR(0, s - 1, 4);
            if (!mbar_wait_warp(&s_full[s & 1], (s >> 1) & 1, ctl, kBSiteSFull)) return false;
            if (tid == 0) SDPA_TR(0, s - 1, 5);
            tc_fence_after();
            const int q0 = (i_start + s % per_head) * 64;
            const uint32_t tS = tmem + lane_base + kColS + (s & 1) * 64 + wg * 32;
            const float4* lse4 = reinterpret_cast<const float4*>(sRows + (s & 1) * 128 + wg * 32);
            const bool need_mask = (p.causal && q0 < kv0 + 128) || (kv0 + 128 > L);
            uint32_t sr[32];
            tmem_ld_x32(tS, sr);
            tmem_wait_ld();
#pragma unroll
            for (int i4 = 0; i4 < 8; ++i4) {
                const float4 l4 = lse4[i4];
                const float lv[4] = {l4.x, l4.y, l4.z, l4.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int i = i4 * 4 + e;
#ifdef SDPA_EXP_NO_EXP
                    float v = fmaf(__uint_as_float(sr[i]), p.scale_log2, -lv[e]) * 1e-3f;
#else
                    float v = fast_exp2(fmaf(__uint_as_float(sr[i]), p.scale_log2, -lv[e]));
#endif
                    if (need_mask) {
                        const int qq = q0 + wg * 32 + i;
                        if (!key_ok || (p.causal && key > qq)) v = 0.f;
                    }
                    pr[i] = v;
                }
            }
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = pack_bf16x2(pr[2 * i], pr[2 * i + 1]);
            tmem_st_x16(tS, pk);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&p_ready[s & 1]);
            if (tid == 0) SDPA_TR(0, s - 1, 6);
            return true;
        };
        // B(s): dS^T = P^T * (dP^T - D_i) -> bf16 -> swizzled shared memory
        auto stage_b = [&](int s) -> bool {
            if (tid == 0) SDPA_TR(0, s, 0);
            if (!mbar_wait_warp(&dp_full[s & 1], (s >> 1) & 1, ctl, kBSiteDpFull)) return false;
            if (tid == 0) SDPA_TR(0, s, 1);
            tc_fence_after();
            const uint32_t tDP = tmem + lane_base + kColDP + (s & 1) * 64 + wg * 32;
            const float4* dl4 = reinterpret_cast<const float4*>(sRows + (s & 1) * 128 + 64 + wg * 32);
            uint32_t dr[32];
            tmem_ld_x32(tDP, dr);
            tmem_wait_ld();
#pragma unroll
            for (int i4 = 0; i4 < 8; ++i4) {
                const float4 d4 = dl4[i4];
                pr[i4 * 4 + 0] *= (__uint_as_float(dr[i4 * 4 + 0]) - d4.x);
                pr[i4 * 4 + 1] *= (__uint_as_float(dr[i4 * 4 + 1]) - d4.y);
                pr[i4 * 4 + 2] *= (__uint_as_float(dr[i4 * 4 + 2]) - d4.z);
                pr[i4 * 4 + 3] *= (__uint_as_float(dr[i4 * 4 + 3]) - d4.w);
            }
            if (s >= 2) {
                if (!mbar_wait_warp(&ds_free[s & 1], ((s >> 1) - 1) & 1, ctl, kBSiteDsFree)) return false;
            }
            if (tid == 0) SDPA_TR(0, s, 2);
            uint8_t* ds_buf = sDS + (s & 1) * 16384;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                uint4 w;
                w.x = pack_bf16x2(pr[ch * 8 + 0], pr[ch * 8 + 1]);
                w.y = pack_bf16x2(pr[ch * 8 + 2], pr[ch * 8 + 3]);
                w.z = pack_bf16x2(pr[ch * 8 + 4], pr[ch * 8 + 5]);
                w.w = pack_bf16x2(pr[ch * 8 + 6], pr[ch * 8 + 7]);
                *reinterpret_cast<uint4*>(ds_buf + sw128_offset(r, wg * 4 + ch)) = w;
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(&ds_ready[s & 1]);
            if (tid == 0) SDPA_TR(0, s, 3);
            return true;
        };

        float pre = load_row(0);
        if (tid < 128) sRows[row_which * 64 + row_qi] = pre;
        pre = load_row(1);
        named_bar_sync(1, 256);
        ok = stage_a(0);
        for (int it = 0; it < n_it && ok; ++it) {
            ok = stage_b(it);
            if (!ok) break;
            if (it + 1 < n_it) {
                if (tid < 128) sRows[((it + 1) & 1) * 128 + row_which * 64 + row_qi] = pre;
                pre = load_row(it + 2);
                named_bar_sync(1, 256);
                ok = stage_a(it + 1);
            }
        }
        if (ok) ok = mbar_wait_warp(dkv_full, 0, ctl, kBSiteDkvFull);
        if (ok) {
            tc_fence_after();
            // group 0 writes dV, group 1 writes dK (scaled)
            const uint32_t tAcc = tmem + lane_base + (wg == 0 ? kColDV : kColDK);
            const float mul = wg == 0 ? 1.0f : p.scale;
            __nv_bfloat16* dst = (wg == 0 ? p.dv : p.dk) + (static_cast<size_t>(r0 + key) * p.Hkv + g) * D;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t a[32];
                tmem_ld_x32(tAcc + c * 32, a);
                tmem_wait_ld();
                if (key_ok) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(a[8 * i + 0]) * mul, __uint_as_float(a[8 * i + 1]) * mul);
                        w.y = pack_bf16x2(__uint_as_float(a[8 * i + 2]) * mul, __uint_as_float(a[8 * i + 3]) * mul);
                        w.z = pack_bf16x2(__uint_as_float(a[8 * i + 4]) * mul, __uint_as_float(a[8 * i + 5]) * mul);
                        w.w = pack_bf16x2(__uint_as_float(a[8 * i + 6]) * mul, __uint_as_float(a[8 * i + 7]) * mul);
                        *reinterpret_cast<uint4*>(dst + c * 32 + i * 8) = w;
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
        for (int it = 0; it < n_it && ok; ++it) {
            const int h = g * G + it / per_head;
            const int q0 = (i_start + it % per_head) * 64;
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
            if (x == 0) bulk_wait_read<0>();  // the previous step's reduce has finished reading the staging buffer
            named_bar_sync(2, 128);
            if (x == 0) SDPA_TR(4, it, 3);
            if (x < D) {
#pragma unroll
                for (int i = 0; i < 32; ++i) sDQ[i * D + x] = __uint_as_float(a0[i]);
#pragma unroll
                for (int i = 0; i < 32; ++i) sDQ[(32 + i) * D + x] = __uint_as_float(a1[i]);
            }
            fence_proxy_async_smem();
            named_bar_sync(2, 128);
            if (x == 0) SDPA_TR(4, it, 4);
            if (x == 0) {
                const int nq = min(64, L - q0);
                float* dst = p.dq_acc + (static_cast<size_t>(h) * p.T + r0 + q0) * D;
                bulk_reduce_add_f32(dst, sDQ, static_cast<uint32_t>(nq) * D * 4u);
                bulk_commit();
            }
            if (x == 0) SDPA_TR(4, it, 5);
        }
        if (x == 0) bulk_wait<0>();
    } else if (warp == 13) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            mbar_arrive_expect_tx(kv_full, 2 * Cfg::kTileBytes);
#pragma unroll
            for (int a = 0; a < D / 64; ++a) {
                tma_load_3d(sK + a * Cfg::kAtomBytes, &map_k, kv_full, a * 64, g, r0 + kv0);
                tma_load_3d(sV + a * Cfg::kAtomBytes, &map_v, kv_full, a * 64, g, r0 + kv0);
            }
            bool ok = true;
            int it = 0;
            for (; it < n_it && ok; ++it) {
                const int st = it % NS;
                ok = mbar_wait(&q_empty[st], ((it / NS) & 1) ^ 1, ctl, kBSiteQEmpty);
                if (!ok) break;
                const int h = g * G + it / per_head;
                const int q0 = (i_start + it % per_head) * 64;
                uint8_t* dst = sQdO + st * Cfg::kStageBytes;
                mbar_arrive_expect_tx(&q_full[st], Cfg::kStageBytes);
#pragma unroll
                for (int a = 0; a < D / 64; ++a) {
                    tma_load_3d(dst + a * Cfg::kStepAtomBytes, &map_q, &q_full[st], a * 64, h, r0 + q0);
                    tma_load_3d(dst + Cfg::kStepBytes + a * Cfg::kStepAtomBytes, &map_do, &q_full[st], a * 64, h,
                                r0 + q0);
                }
            }
            if (!ok) {
                mbar_wait(kv_full, 0, ctl, kBSiteDrain);
                for (int back = 1; back <= NS && back <= it; ++back) {
                    const int i2 = it - back;
                    mbar_wait(&q_full[i2 % NS], (i2 / NS) & 1, ctl, kBSiteDrain);
                }
            }
        }
    } else if (warp == 12 || warp == 14 || warp == 15) {
        // ------------------------------------------------------------ MMA issuers
        // One thread can start a tcgen05.mma only about every 90-100 cycles, so the MMAs of a step are
        // spread over three issuing warps:  warp 12: S^T(i+1), dV(i);  warp 14: dK(i), dP^T(i+1);
        // warp 15: dQ^T(i).  Hazards between warps are all covered by mbarriers (see the header).
        if (elect_one()) {
            constexpr uint32_t idesc_s = make_idesc_bf16(128, 64, false, false);   // S^T, dP^T: keys x 64 queries
            constexpr uint32_t idesc_acc = make_idesc_bf16(128, D, false, true);   // dV, dK: keys x d
            constexpr uint32_t idesc_dq = make_idesc_bf16(128, 64, true, true);    // dQ^T: d x 64 queries
            constexpr uint32_t kLboK = (D == 128) ? Cfg::kAtomBytes : 0;           // D=64: rows 64..127 repeat, unused
            // Descriptors are built once; inside the loops they only advance by constants, because
            // every extra instruction of the issuing thread delays the next tcgen05.mma by several cycles.
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
                if (ok) ok = mbar_wait(&q_full[0], 0, ctl, kBSiteQFull);
                if (ok) {
                    tc_fence_after();
                    issue_s(0, 0);
                    umma_commit(&s_full[0]);
                }
                uint32_t stage = 0, nstage = 1 % NS, nphase = (NS == 1) ? 1u : 0u;  // stage of step it / it+1
                for (int it = 0; it < n_it && ok; ++it) {
                    const uint32_t buf = it & 1, ph = (it >> 1) & 1;
                    SDPA_TR(1, it, 0);
                    if (it + 1 < n_it) {
                        ok = mbar_wait(&q_full[nstage], nphase, ctl, kBSiteQFull);
                        if (!ok) break;
                        SDPA_TR(1, it, 1);
                        tc_fence_after();
                        issue_s(buf ^ 1, nstage);
                        umma_commit(&s_full[buf ^ 1]);
                        SDPA_TR(1, it, 2);
                    }
                    // dV += P^T dO   (P^T from TMEM; the 64 queries of the step are the contraction index)
                    ok = mbar_wait(&p_ready[buf], ph, ctl, kBSitePReady);
                    if (!ok) break;
                    SDPA_TR(1, it, 3);
                    tc_fence_after();
                    {
                        const uint64_t dod = do_mn_desc + stage * kStageStep;
                        const uint32_t a = tmem + kColS + buf * 64;
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            umma_ts(tmem + kColDV, a + (kk >> 1) * 32 + (kk & 1) * 8, dod + static_cast<uint64_t>(kk * (2048 >> 4)),
                                    idesc_acc, (it > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(&q_empty[stage]);
                    SDPA_TR(1, it, 4);
                    stage = nstage;
                    if (++nstage == NS) { nstage = 0; nphase ^= 1; }
                }
                if (ok) umma_commit(dkv_full);
            } else if (warp == 14) {
                const uint64_t v_desc = smem_desc_sw128(smem_u32(sV), 0, 1024);
                const uint64_t do_desc = smem_desc_sw128(smem_u32(sQdO) + Cfg::kStepBytes, 0, 1024);            // K-major B
                const uint64_t q_mn_desc = smem_desc_sw128(smem_u32(sQdO), Cfg::kStepAtomBytes, 1024);           // MN-major B
                const uint64_t ds_desc = smem_desc_sw128(smem_u32(sDS), 0, 1024);                                // K-major A
                auto issue_dp = [&](uint32_t buf, uint32_t stage) {  // dP^T = V dO^T into dP buffer `buf`
                    const uint64_t dd = do_desc + stage * kStageStep;
                    const uint32_t d = tmem + kColDP + buf * 64;
#pragma unroll
                    for (int kk = 0; kk < Cfg::kKSteps; ++kk)
                        umma_ss(d, v_desc + kmaj(kk, Cfg::kAtomBytes), dd + kmaj(kk, Cfg::kStepAtomBytes), idesc_s, kk > 0);
                };
                if (ok) ok = mbar_wait(&q_full[0], 0, ctl, kBSiteQFull);
                if (ok) {
                    tc_fence_after();
                    issue_dp(0, 0);
                    umma_commit(&dp_full[0]);
                }
                uint32_t stage = 0, nstage = 1 % NS, nphase = (NS == 1) ? 1u : 0u;
                for (int it = 0; it < n_it && ok; ++it) {
                    const uint32_t buf = it & 1, ph = (it >> 1) & 1;
                    // dK += dS^T Q
                    SDPA_TR(2, it, 0);
                    ok = mbar_wait(&ds_ready[buf], ph, ctl, kBSiteDsReady);
                    if (!ok) break;
                    SDPA_TR(2, it, 1);
                    tc_fence_after();
                    {
                        const uint64_t dsd = ds_desc + buf * kDsStep;
                        const uint64_t qd = q_mn_desc + stage * kStageStep;
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            umma_ss(tmem + kColDK, dsd + static_cast<uint64_t>(kk * 2), qd + static_cast<uint64_t>(kk * (2048 >> 4)),
                                    idesc_acc, (it > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(&ds_free[buf]);
                    umma_commit(&q_empty[stage]);
                    SDPA_TR(2, it, 2);
                    if (it + 1 < n_it) {
                        ok = mbar_wait(&q_full[nstage], nphase, ctl, kBSiteQFull);
                        if (!ok) break;
                        if (it >= 1) {  // the dQ^T that lived in this buffer has been drained
                            ok = mbar_wait(&dq_empty[buf ^ 1], ph ^ ((it & 1) ? 0u : 1u), ctl, kBSiteDqEmpty);
                            if (!ok) break;
                        }
                        SDPA_TR(2, it, 3);
                        tc_fence_after();
                        issue_dp(buf ^ 1, nstage);
                        umma_commit(&dp_full[buf ^ 1]);
                        SDPA_TR(2, it, 4);
                    }
                    stage = nstage;
                    if (++nstage == NS) { nstage = 0; nphase ^= 1; }
                }
                if (ok) umma_commit(dkv_full);
            } else {
                const uint64_t kt_desc = smem_desc_sw128(smem_u32(sK), kLboK, 1024);                             // MN-major A
                const uint64_t ds_mn_desc = smem_desc_sw128(smem_u32(sDS), 0, 1024);                             // MN-major B
                for (int it = 0; it < n_it && ok; ++it) {
                    const uint32_t buf = it & 1, ph = (it >> 1) & 1;
                    SDPA_TR(3, it, 0);
                    ok = mbar_wait(&ds_ready[buf], ph, ctl, kBSiteDsReady);
                    if (!ok) break;
                    SDPA_TR(3, it, 1);
                    tc_fence_after();
                    // dQ^T = K^T dS^T (overwrites the dP^T buffer of this step)
                    const uint64_t dsd = ds_mn_desc + buf * kDsStep;
                    const uint32_t d = tmem + kColDP + buf * 64;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        umma_ss(d, kt_desc + static_cast<uint64_t>(kk * (2048 >> 4)), dsd + static_cast<uint64_t>(kk * (2048 >> 4)),
                                idesc_dq, kk > 0);
                    umma_commit(&dq_full[buf]);
                    umma_commit(&ds_free[buf]);
                    SDPA_TR(3, it, 2);
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
