// Backward attention kernels for sm_100a.
//
// sdpa_bwd_preprocess_kernel : D_i = rowsum(dO * O) per (token, query head), fp32 [Hq, T]; clears
//                              the fp32 dQ accumulator.
// sdpa_bwd_kernel            : one CTA owns one 128-row key/value tile of one (sequence, kv head) and
//                              loops over the query heads of the group and over the 128-row query
//                              tiles that can see it.  Scores are produced transposed (keys on TMEM
//                              lanes, queries on columns) so that P^T feeds dV += P^T dO straight from
//                              TMEM; dS^T goes through shared memory once and serves both
//                              dK += dS^T Q (as a K-major operand) and dQ = dS K (as an MN-major one).
//                              dK and dV stay in TMEM for the whole CTA; dQ tiles are added into the
//                              fp32 accumulator with coalesced reductions.
// sdpa_bwd_dq_convert_kernel : fp32 dQ accumulator * scale -> bf16.
//
// Roles of sdpa_bwd_kernel (16 warps): warps 0-3 / 4-7 two compute groups (thread = key row, each
// group owns 64 query columns), warps 8-11 dQ reduction group, warp 12 MMA issuer, warp 13 TMA
// producer, warps 14-15 idle.
// TMEM: S^T/P^T [0,128), dP^T then dQ [128,256), dV [256,256+D), dK [384,384+D).
#pragma once
#include "ptx.cuh"

namespace sdpa {

struct BwdParams {
    const int32_t* cu_seqlens;
    const float* lse;    // [Hq, T]
    const float* delta;  // [Hq, T]
    float* dq_acc;       // [T, Hq, D] fp32
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
    static constexpr int kQStages = 2;
    static constexpr int kSmemKV = 2 * kTileBytes;
    static constexpr int kSmemQdO = kQStages * 2 * kTileBytes;
    static constexpr int kSmemDS = 128 * 128 * 2;
    static constexpr int kSmemRows = 2 * 2 * 128 * 4;  // lse / delta rows, double buffered
    static constexpr int kSmemBars = 128;
    // no alignment slack: the dynamic shared window is declared 1024-byte aligned and checked at run time
    static constexpr int kSmemBytes = kSmemKV + kSmemQdO + kSmemDS + kSmemRows + kSmemBars;
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
sdpa_bwd_dq_convert_kernel(const float* __restrict__ dq_acc, __nv_bfloat16* __restrict__ dq, long long n8, float scale) {
    const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n8) return;
    const float4 a = reinterpret_cast<const float4*>(dq_acc)[2 * i];
    const float4 b = reinterpret_cast<const float4*>(dq_acc)[2 * i + 1];
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
    const int n_q = (L + 127) >> 7;
    const int i_start = p.causal ? jt : 0;
    const int per_head = n_q - i_start;
    const int n_it = G * per_head;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = smem_raw;
    if ((smem_u32(smem) & 1023u) != 0u) {  // swizzled tiles need 1024-byte alignment
        if (threadIdx.x == 0) atomicCAS(p.status, 0, kStatusInternal);
        return;
    }
    uint8_t* sK = smem;
    uint8_t* sV = smem + Cfg::kTileBytes;
    uint8_t* sQdO = smem + Cfg::kSmemKV;  // stage s: Q at s*2*tile, dO at s*2*tile + tile
    uint8_t* sDS = sQdO + Cfg::kSmemQdO;
    float* sRows = reinterpret_cast<float*>(sDS + Cfg::kSmemDS);  // [2 buffers][2: lse2, delta][128]
    uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(sRows) + Cfg::kSmemRows);
    uint64_t* kv_full = bars;        // 1
    uint64_t* q_full = bars + 1;     // 2
    uint64_t* q_empty = bars + 3;    // 2
    uint64_t* s_full = bars + 5;
    uint64_t* dp_full = bars + 6;
    uint64_t* p_ready = bars + 7;
    uint64_t* ds_ready = bars + 8;
    uint64_t* ds_free = bars + 9;
    uint64_t* dq_full = bars + 10;
    uint64_t* dq_empty = bars + 11;
    uint64_t* dkv_full = bars + 12;
    uint64_t* drain = bars + 13;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 14);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const WaitCtl ctl{p.status, abort_flag};

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(kv_full, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&q_full[i], 1);
            mbar_init(&q_empty[i], 1);
        }
        mbar_init(s_full, 1);
        mbar_init(dp_full, 1);
        mbar_init(p_ready, 256);
        mbar_init(ds_ready, 256);
        mbar_init(ds_free, 1);
        mbar_init(dq_full, 1);
        mbar_init(dq_empty, 128);
        mbar_init(dkv_full, 1);
        mbar_init(drain, 1);
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
    constexpr uint32_t kColS = 0, kColDP = 128, kColDV = 256, kColDK = 384;

    if (warp < 8) {
        // ------------------------------------------------------------ compute groups
        const int wg = warp >> 2;          // owns query columns [64*wg, 64*wg + 64)
        const int r = tid & 127;           // key row inside the tile
        const int key = kv0 + r;           // key index inside the sequence
        const bool key_ok = key < L;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_base + kColS + wg * 64;
        const uint32_t tDP = tmem + lane_base + kColDP + wg * 64;
        bool ok = true;
        for (int it = 0; it < n_it && ok; ++it) {
            const int hq = it / per_head;
            const int h = g * G + hq;
            const int q0 = (i_start + it % per_head) * 128;
            float* rows = sRows + (it & 1) * 256;
            {
                const int which = tid >> 7, qi = tid & 127;
                const int qrow = q0 + qi;
                float val = which == 0 ? INFINITY : 0.f;
                if (qrow < L) {
                    const size_t idx = static_cast<size_t>(h) * p.T + r0 + qrow;
                    val = which == 0 ? p.lse[idx] * 1.4426950408889634f : p.delta[idx];
                }
                rows[which * 128 + qi] = val;
            }
            named_bar_sync(1, 256);
            const float* lse2 = rows + wg * 64;
            const float* dlt = rows + 128 + wg * 64;

            ok = mbar_wait_warp(s_full, it & 1, ctl, kBSiteSFull);
            if (!ok) break;
            tc_fence_after();
            float pr[64];
            const bool need_mask = (p.causal && q0 < kv0 + 128) || (kv0 + 128 > L);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t sr[32];
                tmem_ld_x32(tS + c * 32, sr);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float e = fast_exp2(fmaf(__uint_as_float(sr[i]), p.scale_log2, -lse2[c * 32 + i]));
                    if (need_mask) {
                        const int qq = q0 + wg * 64 + c * 32 + i;
                        if (!key_ok || (p.causal && key > qq)) e = 0.f;
                    }
                    pr[c * 32 + i] = e;
                }
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) pk[i] = pack_bf16x2(pr[c * 32 + 2 * i], pr[c * 32 + 2 * i + 1]);
                tmem_st_x16(tS + c * 16, pk);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(p_ready);

            ok = mbar_wait_warp(dp_full, it & 1, ctl, kBSiteDpFull);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t dr[32];
                tmem_ld_x32(tDP + c * 32, dr);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) pr[c * 32 + i] *= (__uint_as_float(dr[i]) - dlt[c * 32 + i]);
            }
            if (it > 0) {
                ok = mbar_wait_warp(ds_free, (it - 1) & 1, ctl, kBSiteDsFree);
                if (!ok) break;
            }
            uint8_t* ds_atom = sDS + wg * 16384;
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
                uint4 w;
                w.x = pack_bf16x2(pr[ch * 8 + 0], pr[ch * 8 + 1]);
                w.y = pack_bf16x2(pr[ch * 8 + 2], pr[ch * 8 + 3]);
                w.z = pack_bf16x2(pr[ch * 8 + 4], pr[ch * 8 + 5]);
                w.w = pack_bf16x2(pr[ch * 8 + 6], pr[ch * 8 + 7]);
                *reinterpret_cast<uint4*>(ds_atom + sw128_offset(r, ch)) = w;
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(ds_ready);
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
        const int x = tid & 127;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tDQ = tmem + lane_base + kColDP;
        bool ok = true;
        for (int it = 0; it < n_it && ok; ++it) {
            const int hq = it / per_head;
            const int h = g * G + hq;
            const int q0 = (i_start + it % per_head) * 128;
            ok = mbar_wait_warp(dq_full, it & 1, ctl, kBSiteDqFull);
            if (!ok) break;
            tc_fence_after();
            if constexpr (D == 128) {
                // dQ^T: lane = d, columns = queries; one warp instruction adds 128 contiguous bytes
                float* base = p.dq_acc + (static_cast<size_t>(r0 + q0) * p.Hq + h) * D + x;
                const size_t qstride = static_cast<size_t>(p.Hq) * D;
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t a[32];
                    tmem_ld_x32(tDQ + c * 32, a);
                    tmem_wait_ld();
                    if (c == 3) {
                        tc_fence_before();
                        mbar_arrive(dq_empty);
                    }
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int qq = c * 32 + i;
                        if (q0 + qq < L) atomicAdd(base + qq * qstride, __uint_as_float(a[i]));
                    }
                }
            } else {
                // dQ: lane = query row, columns = d
                const int qq = q0 + x;
                float* base = p.dq_acc + (static_cast<size_t>(r0 + qq) * p.Hq + h) * D;
#pragma unroll 1
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t a[32];
                    tmem_ld_x32(tDQ + c * 32, a);
                    tmem_wait_ld();
                    if (c == D / 32 - 1) {
                        tc_fence_before();
                        mbar_arrive(dq_empty);
                    }
                    if (qq < L) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) atomicAdd(base + c * 32 + i, __uint_as_float(a[i]));
                    }
                }
            }
        }
    } else if (warp == 13) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            auto load_tile = [&](const CUtensorMap* map, uint8_t* dst, uint64_t* bar, int head, int tok) {
#pragma unroll
                for (int a = 0; a < D / 64; ++a) tma_load_3d(dst + a * Cfg::kAtomBytes, map, bar, a * 64, head, tok);
            };
            mbar_arrive_expect_tx(kv_full, 2 * Cfg::kTileBytes);
            load_tile(&map_k, sK, kv_full, g, r0 + kv0);
            load_tile(&map_v, sV, kv_full, g, r0 + kv0);
            bool ok = true;
            int it = 0;
            for (; it < n_it && ok; ++it) {
                const int st = it & 1;
                ok = mbar_wait(&q_empty[st], ((it >> 1) & 1) ^ 1, ctl, kBSiteQEmpty);
                if (!ok) break;
                const int h = g * G + it / per_head;
                const int q0 = (i_start + it % per_head) * 128;
                uint8_t* dst = sQdO + st * 2 * Cfg::kTileBytes;
                mbar_arrive_expect_tx(&q_full[st], 2 * Cfg::kTileBytes);
                load_tile(&map_q, dst, &q_full[st], h, r0 + q0);
                load_tile(&map_do, dst + Cfg::kTileBytes, &q_full[st], h, r0 + q0);
            }
            if (!ok) {
                mbar_wait(kv_full, 0, ctl, kBSiteDrain);
                for (int back = 1; back <= 2 && back <= it; ++back) {
                    const int i2 = it - back;
                    mbar_wait(&q_full[i2 & 1], (i2 >> 1) & 1, ctl, kBSiteDrain);
                }
            }
        }
    } else if (warp == 12) {
        // ------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            constexpr uint32_t idesc_kk = make_idesc_bf16(128, 128, false, false);  // S^T, dP^T
            constexpr uint32_t idesc_kmn = make_idesc_bf16(128, D, false, true);    // dV, dK
            constexpr uint32_t idesc_dq = (D == 128) ? make_idesc_bf16(128, 128, true, true)   // dQ^T = K^T dS^T
                                                     : make_idesc_bf16(128, D, true, true);    // dQ = dS K
            const uint32_t k_addr = smem_u32(sK), v_addr = smem_u32(sV), ds_addr = smem_u32(sDS);
            const uint32_t qdo_addr = smem_u32(sQdO);
            auto kmajor_off = [](int kk) -> uint32_t { return (kk >> 2) * Cfg::kAtomBytes + (kk & 3) * 32; };
            auto issue_st = [&](int st) {  // S^T = K Q^T
                const uint32_t q_addr = qdo_addr + st * 2 * Cfg::kTileBytes;
#pragma unroll
                for (int kk = 0; kk < Cfg::kKSteps; ++kk)
                    umma_ss(tmem + kColS, smem_desc_sw128(k_addr + kmajor_off(kk), 0, 1024),
                            smem_desc_sw128(q_addr + kmajor_off(kk), 0, 1024), idesc_kk, kk > 0);
            };
            bool ok = mbar_wait(kv_full, 0, ctl, kBSiteKvFull);
            if (ok) ok = mbar_wait(&q_full[0], 0, ctl, kBSiteQFull);
            if (ok) {
                tc_fence_after();
                issue_st(0);
                umma_commit(s_full);
            }
            for (int it = 0; it < n_it && ok; ++it) {
                const int st = it & 1;
                const uint32_t q_addr = qdo_addr + st * 2 * Cfg::kTileBytes;
                const uint32_t do_addr = q_addr + Cfg::kTileBytes;
                if (it > 0) {
                    ok = mbar_wait(dq_empty, (it - 1) & 1, ctl, kBSiteDqEmpty);
                    if (!ok) break;
                    tc_fence_after();
                }
                // dP^T = V dO^T
#pragma unroll
                for (int kk = 0; kk < Cfg::kKSteps; ++kk)
                    umma_ss(tmem + kColDP, smem_desc_sw128(v_addr + kmajor_off(kk), 0, 1024),
                            smem_desc_sw128(do_addr + kmajor_off(kk), 0, 1024), idesc_kk, kk > 0);
                umma_commit(dp_full);
                // dV += P^T dO   (P^T from TMEM, queries are the contraction index)
                ok = mbar_wait(p_ready, it & 1, ctl, kBSitePReady);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    umma_ts(tmem + kColDV, tmem + kColS + (kk >> 2) * 64 + (kk & 3) * 8,
                            smem_desc_sw128(do_addr + kk * 2048, Cfg::kAtomBytes, 1024), idesc_kmn,
                            (it > 0 || kk > 0) ? 1u : 0u);
                // next S^T early, so the compute groups can start on it while dK/dQ run
                if (it + 1 < n_it) {
                    const int st2 = (it + 1) & 1;
                    ok = mbar_wait(&q_full[st2], ((it + 1) >> 1) & 1, ctl, kBSiteQFull);
                    if (!ok) break;
                    tc_fence_after();
                    issue_st(st2);
                    umma_commit(s_full);
                }
                ok = mbar_wait(ds_ready, it & 1, ctl, kBSiteDsReady);
                if (!ok) break;
                tc_fence_after();
                // dK += dS^T Q
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    umma_ss(tmem + kColDK, smem_desc_sw128(ds_addr + (kk >> 2) * 16384 + (kk & 3) * 32, 0, 1024),
                            smem_desc_sw128(q_addr + kk * 2048, Cfg::kAtomBytes, 1024), idesc_kmn,
                            (it > 0 || kk > 0) ? 1u : 0u);
                // dQ tile (overwrites the dP^T columns)
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    if constexpr (D == 128)
                        umma_ss(tmem + kColDP, smem_desc_sw128(k_addr + kk * 2048, Cfg::kAtomBytes, 1024),
                                smem_desc_sw128(ds_addr + kk * 2048, 16384, 1024), idesc_dq, kk > 0);
                    else
                        umma_ss(tmem + kColDP, smem_desc_sw128(ds_addr + kk * 2048, 16384, 1024),
                                smem_desc_sw128(k_addr + kk * 2048, Cfg::kAtomBytes, 1024), idesc_dq, kk > 0);
                }
                umma_commit(dq_full);
                umma_commit(&q_empty[st]);
                umma_commit(ds_free);
            }
            if (ok) umma_commit(dkv_full);
            if (!ok) {
                umma_commit(drain);
                mbar_wait(drain, 0, ctl, kBSiteDrain);
            }
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 12) tmem_dealloc(tmem, 512);
}

}  // namespace sdpa
