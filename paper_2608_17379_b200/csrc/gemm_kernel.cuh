// bf16 GEMM C = A B^T for sm_100a (A [M,K], B [N,K], C [M,N], all row-major bf16, fp32 accumulation).
//
// Persistent, warp-specialised kernel, one CTA per SM, output tile 256 x 224:
//   warp 0      TMA producer (one elected lane): A tile 256x64 and B tile 224x64 per k-block into a
//               3-slot mbarrier ring that runs on across output tiles
//   warp 1      MMA issuer (one elected lane): eight tcgen05.mma 128x224x16 per k-block (two 128-row
//               halves sharing the B tile), descriptors built once and advanced by constants; the two
//               accumulators live in TMEM (columns [0,224) and [256,480))
//   warps 4-11  epilogue: TMEM -> registers -> bf16 -> global, one thread per output row
// A 128 x 224 tile per CTA was measured L2-bandwidth-bound (44 KB of operands per 3.7 MFLOP); the
// 256-row tile moves 60 KB per 7.3 MFLOP, a third less, at the price of an epilogue that is not
// overlapped with the next main loop (both accumulators are in use; about 5 % of a tile's time).
// Output tiles are walked in groups of 8 row-tiles so that the A rows and B rows touched by the CTAs
// running at the same time fit the L2.  Tile width 224: the benchmark shape (N = 7168 = 32 * 224) gives
// 1024 tiles = 6.9 rounds of 148 CTAs (98.8 % of the last round used); 256-wide tiles would give 6.05.
#pragma once
#include "ptx.cuh"

namespace sdpa {

struct GemmParams {
    __nv_bfloat16* c;
    int* status;
    int M, N, K;
};

struct GemmCfg {
    static constexpr int kThreads = 384;
    static constexpr int BM = 256, BN = 224, BK = 64;
    static constexpr int kStages = 3;
    static constexpr int kABytes = BM * BK * 2;   // 32 KB
    static constexpr int kBBytes = BN * BK * 2;   // 28 KB
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kGroupM = 8;
    static constexpr int kSmemBars = 256;
    static constexpr int kSmemBytes = kStages * kStageBytes + kSmemBars;  // dynamic window is 1024-aligned (checked)
};

enum GemmSite { kGSiteFull = 41, kGSiteEmpty = 42, kGSiteTmemFull = 43, kGSiteTmemEmpty = 44, kGSiteDrain = 45 };

// 2-D tiled load global -> shared (c0 = innermost coordinate, a multiple of 8 elements for bf16).
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
        : "memory");
}

__global__ void __launch_bounds__(384, 1)
gemm_bf16_nt_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    const GemmParams p) {
    using Cfg = GemmCfg;
    constexpr int S = Cfg::kStages;
    extern __shared__ __align__(1024) uint8_t smem[];
    if ((smem_u32(smem) & 1023u) != 0u) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0, kStatusInternal);
        return;
    }
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S * Cfg::kStageBytes);
    uint64_t* full = bars;                 // [S]
    uint64_t* empty = bars + S;            // [S]
    uint64_t* tmem_full = bars + 2 * S;    // [1]
    uint64_t* tmem_empty = tmem_full + 1;  // [1]
    uint64_t* drain = tmem_empty + 1;      // [1]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5;
    const WaitCtl ctl{p.status, abort_flag};
    const int tiles_m = (p.M + Cfg::BM - 1) / Cfg::BM;
    const int tiles_n = (p.N + Cfg::BN - 1) / Cfg::BN;
    const int n_tiles = tiles_m * tiles_n;
    const int n_kb = (p.K + Cfg::BK - 1) / Cfg::BK;

    // tile index -> (row tile, column tile): groups of kGroupM row tiles, row tile fastest inside a group
    auto tile_coords = [&](int t, int& tm, int& tn) {
        const int per_group = Cfg::kGroupM * tiles_n;
        const int grp = t / per_group;
        const int first = grp * Cfg::kGroupM;
        const int rows_in_group = min(Cfg::kGroupM, tiles_m - first);
        const int r = t - grp * per_group;
        tm = first + r % rows_in_group;
        tn = r / rows_in_group;
    };

    if (tid == 0) {
        *abort_flag = 0;
        for (int i = 0; i < S; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], 1);
        }
        mbar_init(tmem_full, 1);
        mbar_init(tmem_empty, 256);
        mbar_init(drain, 1);
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    if (warp == 0 && elect_one()) {
        prefetch_tmap(&map_a);
        prefetch_tmap(&map_b);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            uint32_t st = 0, ph = 0;
            bool ok = true;
            int issued = 0;
            for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
                int tm, tn;
                tile_coords(t, tm, tn);
                for (int kb = 0; kb < n_kb && ok; ++kb) {
                    ok = mbar_wait(&empty[st], ph ^ 1, ctl, kGSiteEmpty);
                    if (!ok) break;
                    uint8_t* dst = smem + st * Cfg::kStageBytes;
                    mbar_arrive_expect_tx(&full[st], Cfg::kStageBytes);
                    tma_load_2d(dst, &map_a, &full[st], kb * Cfg::BK, tm * Cfg::BM);
                    tma_load_2d(dst + Cfg::kABytes, &map_b, &full[st], kb * Cfg::BK, tn * Cfg::BN);
                    ++issued;
                    if (++st == S) { st = 0; ph ^= 1; }
                }
            }
            if (!ok) {
                // abandon: let the copies already issued land before the CTA exits
                for (int back = 1; back <= S && back <= issued; ++back) {
                    const int i2 = issued - back;
                    mbar_wait(&full[i2 % S], (i2 / S) & 1, ctl, kGSiteDrain);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            constexpr uint32_t idesc = make_idesc_bf16(128, Cfg::BN, false, false);
            constexpr uint64_t kStageStep = Cfg::kStageBytes >> 4;
            constexpr uint64_t kHalfStep = (128 * Cfg::BK * 2) >> 4;  // second 128-row half of the A tile
            const uint64_t a_desc = smem_desc_sw128(smem_u32(smem), 0, 1024);
            const uint64_t b_desc = smem_desc_sw128(smem_u32(smem) + Cfg::kABytes, 0, 1024);
            uint32_t st = 0, ph = 0;
            bool ok = true;
            int local = 0;
            for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++local) {
                // the epilogue has read the previous tile out of the accumulators
                ok = mbar_wait(tmem_empty, (local & 1) ^ 1, ctl, kGSiteTmemEmpty);
                if (!ok) break;
                tc_fence_after();
                for (int kb = 0; kb < n_kb && ok; ++kb) {
                    ok = mbar_wait(&full[st], ph, ctl, kGSiteFull);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t ad = a_desc + st * kStageStep;
                    const uint64_t bd = b_desc + st * kStageStep;
#pragma unroll
                    for (int kk = 0; kk < Cfg::BK / 16; ++kk) {
                        umma_ss(tmem, ad + static_cast<uint64_t>(kk * 2), bd + static_cast<uint64_t>(kk * 2), idesc,
                                (kb > 0 || kk > 0) ? 1u : 0u);
                        umma_ss(tmem + 256, ad + kHalfStep + static_cast<uint64_t>(kk * 2), bd + static_cast<uint64_t>(kk * 2),
                                idesc, (kb > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(&empty[st]);
                    if (++st == S) { st = 0; ph ^= 1; }
                }
                if (ok) umma_commit(tmem_full);
            }
            if (!ok) {
                umma_commit(drain);
                mbar_wait(drain, 0, ctl, kGSiteDrain);
            }
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------ epilogue (thread = output row)
        const int half = (warp - 4) >> 2;                // warps 4-7: rows 0..127, warps 8-11: rows 128..255
        const int row_in_tile = half * 128 + ((tid - 128) & 127);
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        bool ok = true;
        int local = 0;
        for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++local) {
            int tm, tn;
            tile_coords(t, tm, tn);
            ok = mbar_wait_warp(tmem_full, local & 1, ctl, kGSiteTmemFull);
            if (!ok) break;
            tc_fence_after();
            const int row = tm * Cfg::BM + row_in_tile;
            const int col0 = tn * Cfg::BN;
            __nv_bfloat16* crow = p.c + static_cast<size_t>(row) * p.N + col0;
            const uint32_t t_acc = tmem + lane_base + half * 256;
#pragma unroll 1
            for (int c = 0; c < Cfg::BN / 32; ++c) {
                uint32_t r[32];
                tmem_ld_x32(t_acc + c * 32, r);
                tmem_wait_ld();
                if (c == Cfg::BN / 32 - 1) {
                    tc_fence_before();
                    mbar_arrive(tmem_empty);  // accumulator fully read: the next tile may overwrite it
                }
                if (row < p.M) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int col = col0 + c * 32 + i * 8;
                        if (col + 8 <= p.N) {
                            uint4 w;
                            w.x = pack_bf16x2(__uint_as_float(r[8 * i + 0]), __uint_as_float(r[8 * i + 1]));
                            w.y = pack_bf16x2(__uint_as_float(r[8 * i + 2]), __uint_as_float(r[8 * i + 3]));
                            w.z = pack_bf16x2(__uint_as_float(r[8 * i + 4]), __uint_as_float(r[8 * i + 5]));
                            w.w = pack_bf16x2(__uint_as_float(r[8 * i + 6]), __uint_as_float(r[8 * i + 7]));
                            *reinterpret_cast<uint4*>(crow + c * 32 + i * 8) = w;
                        }
                    }
                }
            }
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

}  // namespace sdpa
