// Host side of the C ABI declared in include/sdpa.h: argument checks, TMA tensor maps, launches.
// Links against the CUDA runtime only; cuTensorMapEncodeTiled is fetched through
// cudaGetDriverEntryPoint.  Nothing here allocates or frees device memory.
#include "../../include/sdpa.h"

#include <math.h>
#include <algorithm>
#include <mutex>

#include "bwd_kernel.cuh"
#include "fwd_kernel.cuh"
#include "gemm_kernel.cuh"

namespace sdpa {

__device__ int g_status_word;  // per-device status (0 = ok), latched by the kernels

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static thread_local int tl_last_cuda_error = 0;
// Optional caller-owned events recorded around the main backward kernel (profiling hook).
static thread_local cudaEvent_t tl_ev_main_start = nullptr;
static thread_local cudaEvent_t tl_ev_main_stop = nullptr;

#define SDPA_CUDA_TRY(expr)                          \
    do {                                             \
        cudaError_t e__ = (expr);                    \
        if (e__ != cudaSuccess) {                    \
            tl_last_cuda_error = static_cast<int>(e__); \
            (void)cudaGetLastError();                \
            return SDPA_ERR_CUDA;                    \
        }                                            \
    } while (0)

constexpr int kMaxDevices = 64;
struct DeviceState {
    bool ready = false;
    bool arch_ok = false;
    int* status_ptr = nullptr;
    int num_sms = 0;
};
static DeviceState g_dev[kMaxDevices];
static std::mutex g_mutex;
static EncodeTiledFn g_encode = nullptr;

// Per-device one-time set-up: architecture check, status-word address, shared-memory opt-in.
static int device_state(DeviceState** out) {
    int dev = -1;
    SDPA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SDPA_ERR_ARCH;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState& st = g_dev[dev];
    if (!st.ready) {
        int major = 0;
        SDPA_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        SDPA_CUDA_TRY(cudaDeviceGetAttribute(&st.num_sms, cudaDevAttrMultiProcessorCount, dev));
        st.arch_ok = (major == 10);
        if (st.arch_ok) {
            if (!g_encode) {
                void* fn = nullptr;
                cudaDriverEntryPointQueryResult q;
                SDPA_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
                if (fn == nullptr || q != cudaDriverEntryPointSuccess) {
                    tl_last_cuda_error = static_cast<int>(cudaErrorNotSupported);
                    return SDPA_ERR_CUDA;
                }
                g_encode = reinterpret_cast<EncodeTiledFn>(fn);
            }
            void* sym = nullptr;
            SDPA_CUDA_TRY(cudaGetSymbolAddress(&sym, g_status_word));
            st.status_ptr = static_cast<int*>(sym);
            SDPA_CUDA_TRY(cudaMemset(st.status_ptr, 0, sizeof(int)));
            SDPA_CUDA_TRY(cudaFuncSetAttribute(sdpa_fwd_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               FwdCfg<128>::kSmemBytes));
            SDPA_CUDA_TRY(cudaFuncSetAttribute(sdpa_fwd_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               FwdCfg<64>::kSmemBytes));
            SDPA_CUDA_TRY(cudaFuncSetAttribute(sdpa_fwd_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               FwdCfg<128>::kSmemBytes));
            SDPA_CUDA_TRY(cudaFuncSetAttribute(sdpa_fwd_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               FwdCfg<64>::kSmemBytes));
            SDPA_CUDA_TRY(cudaFuncSetAttribute(sdpa_fwd_kernel<128, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               FwdCfg<128>::kSmemBytes));
            SDPA_CUDA_TRY(cudaFuncSetAttribute(sdpa_fwd_kernel<64, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               FwdCfg<64>::kSmemBytes));
            SDPA_CUDA_TRY(cudaFuncSetAttribute(sdpa_bwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               BwdCfg<128>::kSmemBytes));
            SDPA_CUDA_TRY(cudaFuncSetAttribute(sdpa_bwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               BwdCfg<64>::kSmemBytes));
            SDPA_CUDA_TRY(cudaFuncSetAttribute(gemm_bf16_nt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               GemmCfg::kSmemBytes));
        }
        st.ready = true;
    }
    *out = &st;
    return st.arch_ok ? SDPA_OK : SDPA_ERR_ARCH;
}

// Tensor map over a bf16 attention tensor with H heads, box = box_rows rows of 64 columns, 128B swizzle.
// Packed [T, H, D]: dims {D, H, T, 1}, box {64, 1, rows, 1}.  Dense [B, H, S, D]: dims {D, S, H, B}, box
// {64, rows, 1, 1}.  Both keep the strides increasing and give the same [rows][64] tile in shared memory.
static int make_map(CUtensorMap* map, const void* base, const TensorLayout& lay, int n_batch, int rows, int H, int D,
                    int box_rows, int box_heads = 1) {
    cuuint64_t dims[4], strides[3];
    cuuint32_t box[4];
    const cuuint64_t u = static_cast<cuuint64_t>(D) * 2;
    if (lay.dense) {
        dims[0] = D; dims[1] = rows; dims[2] = H; dims[3] = n_batch;
        strides[0] = u; strides[1] = u * rows; strides[2] = u * rows * H;
        box[0] = 64; box[1] = box_rows; box[2] = box_heads; box[3] = 1;
    } else {
        dims[0] = D; dims[1] = H; dims[2] = rows; dims[3] = 1;
        strides[0] = u; strides[1] = u * H; strides[2] = u * H * rows;
        box[0] = 64; box[1] = box_heads; box[2] = box_rows; box[3] = 1;
    }
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
                                estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        tl_last_cuda_error = static_cast<int>(r);
        return SDPA_ERR_CUDA;
    }
    return SDPA_OK;
}

static TensorLayout packed_layout(int T, int Hq, int Hkv, int D) {
    TensorLayout l{};
    l.ts_q = Hq * D; l.hs_q = D; l.ts_kv = Hkv * D; l.hs_kv = D;
    l.lse_hs = T; l.lse_bs = 0; l.bs_q = 0; l.bs_kv = 0;
    l.dense = 0; l.S = T > 0 ? T : 1; l.has_lengths = 1;
    return l;
}
static TensorLayout dense_layout(int Hq, int Hkv, int S, int D, bool has_lengths) {
    TensorLayout l{};
    l.ts_q = D; l.hs_q = S * D; l.ts_kv = D; l.hs_kv = S * D;
    l.bs_q = static_cast<long long>(Hq) * S * D; l.bs_kv = static_cast<long long>(Hkv) * S * D;
    l.lse_hs = S; l.lse_bs = static_cast<long long>(Hq) * S;
    l.dense = 1; l.S = S; l.has_lengths = has_lengths ? 1 : 0;
    return l;
}

// Head dimension the kernels are instantiated for: 64 or 128; a smaller head dimension runs in the next
// larger kernel, its missing columns zero-filled by the TMA loads (out-of-bounds box columns read as 0).
static int padded_head_dim(int D) { return D <= 64 ? 64 : 128; }

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_common(const int32_t* cu, int B, int Hq, int Hkv, int D, float scale, int T, int max_seqlen,
                        bool cu_optional = false) {
    if (cu == nullptr && !cu_optional) return SDPA_ERR_NULL;
    if (B < 1 || Hq < 1 || Hkv < 1 || T < 0 || max_seqlen < 0) return SDPA_ERR_SHAPE;
    if (D < 8 || D > 128 || (D % 8) != 0) return SDPA_ERR_SHAPE;
    if (Hq % Hkv != 0) return SDPA_ERR_SHAPE;
    if (!(scale > 0.f) || !isfinite(scale)) return SDPA_ERR_SHAPE;
    if (max_seqlen > T) return SDPA_ERR_SHAPE;
    if (static_cast<long long>(B) * Hq > 2147483647ll) return SDPA_ERR_SHAPE;
    return SDPA_OK;
}

// Forward launch order: how many (sequence, query head) pairs have their CTAs interleaved.  When all K/V
// rows fit the L2 comfortably every pair is interleaved (heaviest query tiles of all heads first, the best
// balance); otherwise a chunk covers as many kv heads as keep about 48 MB of K/V in flight, so that the
// query tiles of one head re-read its K/V from the L2 instead of from DRAM.
static int fwd_head_chunk(int B, int Hq, int Hkv, int D, long long kv_rows) {
    const long long kL2Budget = 48ll << 20;
    const long long total = kv_rows * Hkv * D * 4;  // K and V, bf16
    const int all = B * Hq;
    if (total <= kL2Budget || B <= 0) return all;
    const long long per_kv_head = std::max<long long>(1, kv_rows / B * D * 4);
    const long long kv_heads = std::max<long long>(1, kL2Budget / per_kv_head);
    long long chunk = kv_heads * (Hq / Hkv);
    chunk = std::max<long long>(chunk, (all + 65534) / 65535);  // the chunks are the grid's y dimension
    return static_cast<int>(std::min<long long>(all, chunk));
}

// Backward launch order: how many (sequence, kv head) groups have their CTAs interleaved.  A small dQ
// accumulator stays in the L2 whatever the order, so all groups are interleaved (heaviest key tiles first).
// Otherwise a chunk holds about two waves of CTAs (at least 8 groups), in equal chunks: the CTAs running
// at one time then reduce into few heads' accumulator rows, which stay in the L2 between their visits.
static int bwd_group_chunk(int n_groups, int n_kv_tiles, long long dq_acc_bytes) {
    if (dq_acc_bytes <= (48ll << 20) || n_groups <= 8) return std::max(1, n_groups);
    const int c0 = std::max(8, (296 + n_kv_tiles - 1) / std::max(1, n_kv_tiles));
    const int n_chunks = std::min((n_groups + c0 - 1) / c0, 65535);  // the chunks are the grid's y dimension
    return (n_groups + n_chunks - 1) / n_chunks;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static size_t bwd_dq_bytes(int Hq, int D, int T) { return align_up(static_cast<size_t>(T) * Hq * D * sizeof(float), 256); }
static size_t bwd_delta_bytes(int Hq, int T) { return align_up(static_cast<size_t>(T) * Hq * sizeof(float), 256); }

}  // namespace sdpa

using namespace sdpa;

// Key side of a call whose sequences have their own key row ranges (packed layout only); cu == nullptr: the
// keys of a sequence are the rows of its queries.
struct KeySide {
    const int32_t* cu = nullptr;
    int total = 0;
    int max_seqlen = 0;
};
static int check_key_side(const KeySide& ks, const TensorLayout& lay) {
    if (ks.cu == nullptr) return SDPA_OK;
    if (lay.dense) return SDPA_ERR_SHAPE;
    if (ks.total < 0 || ks.max_seqlen < 0 || ks.max_seqlen > ks.total) return SDPA_ERR_SHAPE;
    return SDPA_OK;
}

static int fwd_launch(const void* q, const void* k, const void* v, void* o, float* lse, const int32_t* cu_seqlens,
                      int B, int Hq, int Hkv, int D, int causal, float scale, int total_tokens, int max_seqlen,
                      void* stream, const TensorLayout& lay, const KeySide& ks = KeySide()) {
    int rc = check_common(cu_seqlens, B, Hq, Hkv, D, scale, total_tokens, max_seqlen, lay.dense != 0);
    if (rc != SDPA_OK) return rc;
    if ((rc = check_key_side(ks, lay)) != SDPA_OK) return rc;
    if (total_tokens == 0 || max_seqlen == 0) return SDPA_OK;
    if (!q || !k || !v || !o || !lse) return SDPA_ERR_NULL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || (reinterpret_cast<uintptr_t>(lse) & 3u))
        return SDPA_ERR_ALIGN;
    DeviceState* st = nullptr;
    rc = device_state(&st);
    if (rc != SDPA_OK) return rc;

    CUtensorMap mq, mk, mv;
    const int map_rows = lay.dense ? lay.S : total_tokens;
    const int key_rows = ks.cu != nullptr ? ks.total : map_rows;
    if (key_rows == 0) return SDPA_ERR_SHAPE;  // queries without any key row
    if ((rc = make_map(&mq, q, lay, B, map_rows, Hq, D, 128)) != SDPA_OK) return rc;
    if ((rc = make_map(&mk, k, lay, B, key_rows, Hkv, D, 128)) != SDPA_OK) return rc;
    if ((rc = make_map(&mv, v, lay, B, key_rows, Hkv, D, 128)) != SDPA_OK) return rc;

    FwdParams p;
    p.lay = lay;
    p.cu_seqlens = cu_seqlens;
    p.cu_seqlens_k = ks.cu;
    p.Tk = ks.total;
    p.part_o = nullptr; p.part_lse = nullptr;
    p.kv_indptr = nullptr; p.kv_indices = nullptr; p.k_cache = nullptr; p.v_cache = nullptr; p.num_pages = 0;
    p.o = static_cast<__nv_bfloat16*>(o);
    p.lse = lse;
    p.status = st->status_ptr;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.T = total_tokens;
    p.causal = causal ? 1 : 0;
    p.max_seqlen = max_seqlen;
    p.d = D;
    p.scale = scale;
    p.scale_log2 = scale * 1.4426950408889634f;
    const int n_pairs = (max_seqlen + 255) / 256;
    if (n_pairs > 65535) return SDPA_ERR_SHAPE;
    p.head_chunk = fwd_head_chunk(B, Hq, Hkv, D, key_rows);
    if (static_cast<long long>(n_pairs) * p.head_chunk > 0x7fffffffLL) return SDPA_ERR_SHAPE;
    dim3 grid(static_cast<unsigned>(n_pairs * p.head_chunk),
              static_cast<unsigned>((B * Hq + p.head_chunk - 1) / p.head_chunk), 1);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (padded_head_dim(D) == 128)
        sdpa_fwd_kernel<128, false><<<grid, FwdCfg<128>::kThreads, FwdCfg<128>::kSmemBytes, s>>>(mq, mk, mv, p);
    else
        sdpa_fwd_kernel<64, false><<<grid, FwdCfg<64>::kThreads, FwdCfg<64>::kSmemBytes, s>>>(mq, mk, mv, p);
    SDPA_CUDA_TRY(cudaGetLastError());
    return SDPA_OK;
}

extern "C" int sdpa_fwd(const void* q, const void* k, const void* v, void* o, float* lse, const int32_t* cu_seqlens,
                        int B, int Hq, int Hkv, int D, int causal, float scale, int total_tokens, int max_seqlen,
                        void* stream) {
    return fwd_launch(q, k, v, o, lse, cu_seqlens, B, Hq, Hkv, D, causal, scale, total_tokens, max_seqlen, stream,
                      packed_layout(total_tokens, Hq, Hkv, D));
}

extern "C" int sdpa_fwd_varlen_qk(const void* q, const void* k, const void* v, void* o, float* lse,
                                  const int32_t* cu_seqlens_q, const int32_t* cu_seqlens_k, int B, int Hq, int Hkv,
                                  int D, int causal, float scale, int total_q, int total_k, int max_seqlen_q,
                                  int max_seqlen_k, void* stream) {
    if (cu_seqlens_k == nullptr) return SDPA_ERR_NULL;
    KeySide ks;
    ks.cu = cu_seqlens_k; ks.total = total_k; ks.max_seqlen = max_seqlen_k;
    return fwd_launch(q, k, v, o, lse, cu_seqlens_q, B, Hq, Hkv, D, causal, scale, total_q, max_seqlen_q, stream,
                      packed_layout(total_q, Hq, Hkv, D), ks);
}

// Limits of the dense entry points: B * S rows are indexed with 32-bit integers.
static int check_dense(int B, int S) {
    if (B < 1 || S < 0) return SDPA_ERR_SHAPE;
    if (static_cast<long long>(B) * S > 2147483647ll) return SDPA_ERR_SHAPE;
    return SDPA_OK;
}

extern "C" int sdpa_fwd_bhsd(const void* q, const void* k, const void* v, void* o, float* lse,
                             const int32_t* cu_seqlens, int B, int Hq, int Hkv, int S, int D, int causal, float scale,
                             void* stream) {
    const int rc = check_dense(B, S);
    if (rc != SDPA_OK) return rc;
    return fwd_launch(q, k, v, o, lse, cu_seqlens, B, Hq, Hkv, D, causal, scale, B * S, S, stream,
                      dense_layout(Hq, Hkv, S, D, cu_seqlens != nullptr));
}

extern "C" int sdpa_fwd_paged(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                              const int32_t* cu_seqlens_q, const int32_t* kv_indptr, const int32_t* kv_indices, int B,
                              int Hq, int Hkv, int D, int causal, float scale, int total_q, int max_seqlen_q,
                              int num_pages, void* stream) {
    int rc = check_common(cu_seqlens_q, B, Hq, Hkv, D, scale, total_q, max_seqlen_q);
    if (rc != SDPA_OK) return rc;
    if (num_pages < 0) return SDPA_ERR_SHAPE;
    if (total_q == 0 || max_seqlen_q == 0) return SDPA_OK;
    if (!q || !k_cache || !v_cache || !o || !lse || !kv_indptr || !kv_indices) return SDPA_ERR_NULL;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(o) ||
        (reinterpret_cast<uintptr_t>(lse) & 3u))
        return SDPA_ERR_ALIGN;
    if (num_pages == 0) return SDPA_ERR_SHAPE;
    DeviceState* st = nullptr;
    rc = device_state(&st);
    if (rc != SDPA_OK) return rc;
    CUtensorMap mq;
    const TensorLayout lay = packed_layout(total_q, Hq, Hkv, D);
    if ((rc = make_map(&mq, q, lay, 1, total_q, Hq, D, 128)) != SDPA_OK) return rc;
    FwdParams p;
    p.lay = lay;
    p.cu_seqlens_k = nullptr;
    p.Tk = 0;
    p.part_o = nullptr; p.part_lse = nullptr;
    p.cu_seqlens = cu_seqlens_q;
    p.kv_indptr = kv_indptr;
    p.kv_indices = kv_indices;
    p.k_cache = static_cast<const __nv_bfloat16*>(k_cache);
    p.v_cache = static_cast<const __nv_bfloat16*>(v_cache);
    p.num_pages = num_pages;
    p.o = static_cast<__nv_bfloat16*>(o);
    p.lse = lse;
    p.status = st->status_ptr;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.T = total_q;
    p.causal = causal ? 1 : 0;
    p.max_seqlen = max_seqlen_q;
    p.d = D;
    p.scale = scale;
    p.scale_log2 = scale * 1.4426950408889634f;
    const int n_pairs = (max_seqlen_q + 255) / 256;
    if (n_pairs > 65535) return SDPA_ERR_SHAPE;
    p.head_chunk = fwd_head_chunk(B, Hq, Hkv, D, num_pages);
    if (static_cast<long long>(n_pairs) * p.head_chunk > 0x7fffffffLL) return SDPA_ERR_SHAPE;
    dim3 grid(static_cast<unsigned>(n_pairs * p.head_chunk),
              static_cast<unsigned>((B * Hq + p.head_chunk - 1) / p.head_chunk), 1);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the K/V tensor maps are unused by the gathering producer; the Q map stands in for them
    if (padded_head_dim(D) == 128)
        sdpa_fwd_kernel<128, true><<<grid, FwdCfg<128>::kThreads, FwdCfg<128>::kSmemBytes, s>>>(mq, mq, mq, p);
    else
        sdpa_fwd_kernel<64, true><<<grid, FwdCfg<64>::kThreads, FwdCfg<64>::kSmemBytes, s>>>(mq, mq, mq, p);
    SDPA_CUDA_TRY(cudaGetLastError());
    return SDPA_OK;
}

// Decode path: key tiles per CTA and the number of key splits that follows for the longest sequence.  Every
// CTA takes the same number of tiles, so short sequences use fewer CTAs (their surplus splits leave at once).
// A CTA costs about 5 us before its first tile is done, so CTAs are kept long: at least 8 tiles, and enough
// that all (sequence, kv head) groups at full length would fit one wave of a B200's 148 SMs.
static int decode_tiles_per_split(int B, int Hkv, int max_seqlen_k) {
    const long long tiles = std::max(1, (max_seqlen_k + 127) / 128);
    const long long one_wave = (tiles * B * Hkv + 147) / 148;
    return static_cast<int>(std::max<long long>(1, std::min<long long>(std::max<long long>(8, one_wave), tiles)));
}
static int decode_splits(int B, int Hkv, int max_seqlen_k) {
    const int tiles = std::max(1, (max_seqlen_k + 127) / 128);
    const int tps = decode_tiles_per_split(B, Hkv, max_seqlen_k);
    return (tiles + tps - 1) / tps;
}

extern "C" size_t sdpa_decode_paged_workspace_bytes(int B, int Hq, int Hkv, int D, int max_seqlen_k) {
    if (B < 1 || Hq < 1 || Hkv < 1 || max_seqlen_k < 0 || D < 8 || D > 128 || (D % 8) != 0 || Hq % Hkv != 0) return 0;
    const size_t rows = static_cast<size_t>(2 * decode_splits(B, Hkv, max_seqlen_k)) * B * Hq;  // two slots per split
    return align_up(rows * D * sizeof(float), 256) + align_up(rows * sizeof(float), 256);
}

extern "C" int sdpa_decode_paged(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                                 const int32_t* kv_indptr, const int32_t* kv_indices, int B, int Hq, int Hkv, int D,
                                 float scale, int max_seqlen_k, int num_pages, void* workspace, size_t workspace_bytes,
                                 void* stream) {
    if (B < 1 || Hq < 1 || Hkv < 1 || max_seqlen_k < 0 || num_pages < 0) return SDPA_ERR_SHAPE;
    if (D < 8 || D > 128 || (D % 8) != 0 || Hq % Hkv != 0 || Hq / Hkv > 128) return SDPA_ERR_SHAPE;
    if (!(scale > 0.f) || !isfinite(scale)) return SDPA_ERR_SHAPE;
    if (!q || !k_cache || !v_cache || !o || !lse || !kv_indptr || !kv_indices) return SDPA_ERR_NULL;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(o) ||
        (reinterpret_cast<uintptr_t>(lse) & 3u))
        return SDPA_ERR_ALIGN;
    if (num_pages == 0 || max_seqlen_k == 0) return SDPA_ERR_SHAPE;  // every query needs at least one key
    const size_t need = sdpa_decode_paged_workspace_bytes(B, Hq, Hkv, D, max_seqlen_k);
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < need)
        return SDPA_ERR_WORKSPACE;
    DeviceState* st = nullptr;
    int rc = device_state(&st);
    if (rc != SDPA_OK) return rc;
    const int G = Hq / Hkv;
    const int n_splits = decode_splits(B, Hkv, max_seqlen_k);
    const TensorLayout lay = packed_layout(B, Hq, Hkv, D);
    CUtensorMap mq;  // box: the G heads of a group for one token
    if ((rc = make_map(&mq, q, lay, 1, B, Hq, D, 1, G)) != SDPA_OK) return rc;
    FwdParams p;
    p.lay = lay;
    p.cu_seqlens = nullptr; p.cu_seqlens_k = nullptr; p.Tk = 0;
    p.kv_indptr = kv_indptr;
    p.kv_indices = kv_indices;
    p.k_cache = static_cast<const __nv_bfloat16*>(k_cache);
    p.v_cache = static_cast<const __nv_bfloat16*>(v_cache);
    p.num_pages = num_pages;
    p.o = static_cast<__nv_bfloat16*>(o);
    p.lse = lse;
    p.status = st->status_ptr;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.T = B;
    p.causal = 0;  // a single query token sees every key of its sequence
    p.max_seqlen = 1;
    p.d = D;
    p.scale = scale;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.head_chunk = 1;
    p.tiles_per_split = decode_tiles_per_split(B, Hkv, max_seqlen_k);
    const size_t rows = static_cast<size_t>(2 * n_splits) * B * Hq;  // every CTA leaves two partial results
    p.part_o = static_cast<float*>(workspace);
    p.part_lse = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + align_up(rows * D * sizeof(float), 256));
    if (static_cast<long long>(B) * Hkv > 2147483647ll) return SDPA_ERR_SHAPE;
    dim3 grid(static_cast<unsigned>(B * Hkv), static_cast<unsigned>(n_splits), 1);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (padded_head_dim(D) == 128)
        sdpa_fwd_kernel<128, true, true><<<grid, FwdCfg<128>::kThreads, FwdCfg<128>::kSmemBytes, s>>>(mq, mq, mq, p);
    else
        sdpa_fwd_kernel<64, true, true><<<grid, FwdCfg<64>::kThreads, FwdCfg<64>::kSmemBytes, s>>>(mq, mq, mq, p);
    SDPA_CUDA_TRY(cudaGetLastError());
    sdpa_decode_combine_kernel<<<static_cast<unsigned>(B * Hq), 32, 0, s>>>(
        p.part_o, p.part_lse, static_cast<__nv_bfloat16*>(o), lse, 2 * n_splits, B, Hq, D);
    SDPA_CUDA_TRY(cudaGetLastError());
    return SDPA_OK;
}

extern "C" size_t sdpa_bwd_workspace_bytes(int B, int Hq, int Hkv, int D, int total_tokens, int max_seqlen) {
    if (B < 1 || Hq < 1 || Hkv < 1 || total_tokens < 0 || max_seqlen < 0 || D < 8 || D > 128 || (D % 8) != 0 || Hq % Hkv != 0)
        return 0;
    // fp32 dQ accumulator, D_i rows, turn counters of the deterministic mode (same size as the D_i rows)
    return bwd_dq_bytes(Hq, padded_head_dim(D), total_tokens) + 2 * bwd_delta_bytes(Hq, total_tokens) + 256;
}

static int bwd_launch(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* dout,
                      void* dq, void* dk, void* dv, const int32_t* cu_seqlens, int B, int Hq, int Hkv, int D,
                      int causal, float scale, int total_tokens, int max_seqlen, void* workspace,
                      size_t workspace_bytes, void* stream, const TensorLayout& lay, bool deterministic = false,
                      const KeySide& ks = KeySide()) {
    int rc = check_common(cu_seqlens, B, Hq, Hkv, D, scale, total_tokens, max_seqlen, lay.dense != 0);
    if (rc != SDPA_OK) return rc;
    if ((rc = check_key_side(ks, lay)) != SDPA_OK) return rc;
    if (total_tokens == 0 || max_seqlen == 0) {
        // no queries at all: keys that exist on their own get zero gradients
        if (ks.cu != nullptr && ks.total > 0) {
            if (!dk || !dv) return SDPA_ERR_NULL;
            const size_t bytes = static_cast<size_t>(ks.total) * Hkv * D * 2;
            SDPA_CUDA_TRY(cudaMemsetAsync(dk, 0, bytes, static_cast<cudaStream_t>(stream)));
            SDPA_CUDA_TRY(cudaMemsetAsync(dv, 0, bytes, static_cast<cudaStream_t>(stream)));
        }
        return SDPA_OK;
    }
    if (!q || !k || !v || !o || !lse || !dout || !dq || !dk || !dv) return SDPA_ERR_NULL;
    if (ks.cu != nullptr && ks.total == 0) return SDPA_ERR_SHAPE;  // queries without any key row
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(dout) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv) || (reinterpret_cast<uintptr_t>(lse) & 3u))
        return SDPA_ERR_ALIGN;
    const size_t need = sdpa_bwd_workspace_bytes(B, Hq, Hkv, D, total_tokens, max_seqlen);
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < need)
        return SDPA_ERR_WORKSPACE;
    DeviceState* st = nullptr;
    rc = device_state(&st);
    if (rc != SDPA_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    float* dq_acc = static_cast<float*>(workspace);
    const int Dp = padded_head_dim(D);
    float* delta = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + bwd_dq_bytes(Hq, Dp, total_tokens));
    int* dq_turn = deterministic ? reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(delta) + bwd_delta_bytes(Hq, total_tokens))
                                 : nullptr;

    // B0: D_i = rowsum(dO * O), and clear the fp32 dQ accumulator.
    {
        const long long rows = static_cast<long long>(total_tokens) * Hq;
        const int threads = 256;
        const int rows_per_block = threads / (Dp / 8);
        const long long blocks = (rows + rows_per_block - 1) / rows_per_block;
        if (Dp == 128)
            sdpa_bwd_preprocess_kernel<128><<<static_cast<unsigned>(blocks), threads, 0, s>>>(
                static_cast<const __nv_bfloat16*>(o), static_cast<const __nv_bfloat16*>(dout), delta, dq_acc, dq_turn,
                total_tokens, Hq, D, lay);
        else
            sdpa_bwd_preprocess_kernel<64><<<static_cast<unsigned>(blocks), threads, 0, s>>>(
                static_cast<const __nv_bfloat16*>(o), static_cast<const __nv_bfloat16*>(dout), delta, dq_acc, dq_turn,
                total_tokens, Hq, D, lay);
        SDPA_CUDA_TRY(cudaGetLastError());
    }

    CUtensorMap mq, mk, mv, mdo;
    const int map_rows = lay.dense ? lay.S : total_tokens;
    const int key_rows = ks.cu != nullptr ? ks.total : map_rows;
    if ((rc = make_map(&mq, q, lay, B, map_rows, Hq, D, 64)) != SDPA_OK) return rc;
    if ((rc = make_map(&mk, k, lay, B, key_rows, Hkv, D, 128)) != SDPA_OK) return rc;
    if ((rc = make_map(&mv, v, lay, B, key_rows, Hkv, D, 128)) != SDPA_OK) return rc;
    if ((rc = make_map(&mdo, dout, lay, B, map_rows, Hq, D, 64)) != SDPA_OK) return rc;

    BwdParams p;
    p.lay = lay;
    p.cu_seqlens = cu_seqlens;
    p.cu_seqlens_k = ks.cu;
    p.Tk = ks.total;
    p.lse = lse;
    p.delta = delta;
    p.dq_acc = dq_acc;
    p.dq_turn = dq_turn;
    p.dk = static_cast<__nv_bfloat16*>(dk);
    p.dv = static_cast<__nv_bfloat16*>(dv);
    p.status = st->status_ptr;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.T = total_tokens;
    p.causal = causal ? 1 : 0;
    p.max_seqlen = max_seqlen;
    p.scale = scale;
    p.scale_log2 = scale * 1.4426950408889634f;
    const int n_kv_tiles = ((ks.cu != nullptr ? ks.max_seqlen : max_seqlen) + 127) / 128;
    if (n_kv_tiles > 65535) return SDPA_ERR_SHAPE;
    // x walks a chunk of (sequence, kv head) groups key tile by key tile, y walks the chunks
    const int n_groups = B * Hkv;
    p.d = D;
    p.group_chunk = bwd_group_chunk(n_groups, n_kv_tiles, static_cast<long long>(total_tokens) * Hq * Dp * 4);
    if (static_cast<long long>(n_kv_tiles) * p.group_chunk > 0x7fffffffLL) return SDPA_ERR_SHAPE;
    dim3 grid(static_cast<unsigned>(n_kv_tiles * p.group_chunk),
              static_cast<unsigned>((n_groups + p.group_chunk - 1) / p.group_chunk), 1);
    if (tl_ev_main_start) SDPA_CUDA_TRY(cudaEventRecord(tl_ev_main_start, s));
    if (Dp == 128)
        sdpa_bwd_kernel<128><<<grid, BwdCfg<128>::kThreads, BwdCfg<128>::kSmemBytes, s>>>(mq, mk, mv, mdo, p);
    else
        sdpa_bwd_kernel<64><<<grid, BwdCfg<64>::kThreads, BwdCfg<64>::kSmemBytes, s>>>(mq, mk, mv, mdo, p);
    SDPA_CUDA_TRY(cudaGetLastError());
    if (tl_ev_main_stop) SDPA_CUDA_TRY(cudaEventRecord(tl_ev_main_stop, s));

    // B7 (dQ part): fp32 accumulator -> bf16 with the softmax scale applied.
    {
        const long long n8 = static_cast<long long>(total_tokens) * Hq * D / 8;
        const int threads = 256;
        const long long blocks = (n8 + threads - 1) / threads;
        sdpa_bwd_dq_convert_kernel<<<static_cast<unsigned>(blocks), threads, 0, s>>>(
            dq_acc, static_cast<__nv_bfloat16*>(dq), n8, scale, total_tokens, Hq, Dp, D, lay);
        SDPA_CUDA_TRY(cudaGetLastError());
    }
    return SDPA_OK;
}

extern "C" int sdpa_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* dout,
                        void* dq, void* dk, void* dv, const int32_t* cu_seqlens, int B, int Hq, int Hkv, int D,
                        int causal, float scale, int total_tokens, int max_seqlen, void* workspace,
                        size_t workspace_bytes, void* stream) {
    return bwd_launch(q, k, v, o, lse, dout, dq, dk, dv, cu_seqlens, B, Hq, Hkv, D, causal, scale, total_tokens,
                      max_seqlen, workspace, workspace_bytes, stream, packed_layout(total_tokens, Hq, Hkv, D));
}

extern "C" int sdpa_bwd_varlen_qk(const void* q, const void* k, const void* v, const void* o, const float* lse,
                                  const void* dout, void* dq, void* dk, void* dv, const int32_t* cu_seqlens_q,
                                  const int32_t* cu_seqlens_k, int B, int Hq, int Hkv, int D, int causal, float scale,
                                  int total_q, int total_k, int max_seqlen_q, int max_seqlen_k, void* workspace,
                                  size_t workspace_bytes, void* stream) {
    if (cu_seqlens_k == nullptr) return SDPA_ERR_NULL;
    KeySide ks;
    ks.cu = cu_seqlens_k; ks.total = total_k; ks.max_seqlen = max_seqlen_k;
    return bwd_launch(q, k, v, o, lse, dout, dq, dk, dv, cu_seqlens_q, B, Hq, Hkv, D, causal, scale, total_q,
                      max_seqlen_q, workspace, workspace_bytes, stream, packed_layout(total_q, Hq, Hkv, D), false, ks);
}

extern "C" int sdpa_bwd_deterministic(const void* q, const void* k, const void* v, const void* o, const float* lse,
                                      const void* dout, void* dq, void* dk, void* dv, const int32_t* cu_seqlens, int B,
                                      int Hq, int Hkv, int D, int causal, float scale, int total_tokens, int max_seqlen,
                                      void* workspace, size_t workspace_bytes, void* stream) {
    return bwd_launch(q, k, v, o, lse, dout, dq, dk, dv, cu_seqlens, B, Hq, Hkv, D, causal, scale, total_tokens,
                      max_seqlen, workspace, workspace_bytes, stream, packed_layout(total_tokens, Hq, Hkv, D), true);
}

extern "C" int sdpa_bwd_bhsd(const void* q, const void* k, const void* v, const void* o, const float* lse,
                             const void* dout, void* dq, void* dk, void* dv, const int32_t* cu_seqlens, int B, int Hq,
                             int Hkv, int S, int D, int causal, float scale, void* workspace, size_t workspace_bytes,
                             void* stream) {
    const int rc = check_dense(B, S);
    if (rc != SDPA_OK) return rc;
    return bwd_launch(q, k, v, o, lse, dout, dq, dk, dv, cu_seqlens, B, Hq, Hkv, D, causal, scale, B * S, S,
                      workspace, workspace_bytes, stream, dense_layout(Hq, Hkv, S, D, cu_seqlens != nullptr));
}

// ------------------------------------------------------------------ built-in scratch (no allocation)
// Scratch for sdpa_bwd_static_scratch.  It lives in the library image, so a GPU that loads the
// library keeps these bytes until the process ends.
static __device__ __align__(256) unsigned char g_static_scratch[SDPA_STATIC_SCRATCH_BYTES];
// In host code the name g_static_scratch only stands for the symbol; it is not an address the GPU
// can use.  The real device address differs per device and is looked up once per device below.
static void* g_static_scratch_addr[sdpa::kMaxDevices];

static int static_scratch_address(void** out) {
    int dev = -1;
    SDPA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= sdpa::kMaxDevices) return SDPA_ERR_ARCH;
    std::lock_guard<std::mutex> lock(sdpa::g_mutex);
    if (g_static_scratch_addr[dev] == nullptr) {
        void* addr = nullptr;
        SDPA_CUDA_TRY(cudaGetSymbolAddress(&addr, g_static_scratch));  // for the device that is current now
        if (addr == nullptr) {
            sdpa::tl_last_cuda_error = static_cast<int>(cudaErrorInvalidSymbol);
            return SDPA_ERR_CUDA;
        }
        g_static_scratch_addr[dev] = addr;
    }
    *out = g_static_scratch_addr[dev];
    return SDPA_OK;
}

extern "C" int sdpa_bwd_static_scratch(const void* q, const void* k, const void* v, const void* o, const float* lse,
                                       const void* dout, void* dq, void* dk, void* dv, const int32_t* cu_seqlens,
                                       int B, int Hq, int Hkv, int D, int causal, float scale, int total_tokens,
                                       int max_seqlen, void* stream) {
    int rc = check_common(cu_seqlens, B, Hq, Hkv, D, scale, total_tokens, max_seqlen);
    if (rc != SDPA_OK) return rc;
    if (total_tokens == 0 || max_seqlen == 0) return SDPA_OK;
    const size_t need = sdpa_bwd_workspace_bytes(B, Hq, Hkv, D, total_tokens, max_seqlen);
    if (need == 0 || need > static_cast<size_t>(SDPA_STATIC_SCRATCH_BYTES)) return SDPA_ERR_STATIC_SCRATCH;
    void* scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc != SDPA_OK) return rc;
    // sdpa_bwd clears the dQ accumulator inside the scratch before it accumulates into it and
    // overwrites the D_i rows, so nothing of an earlier call survives into this one.
    return sdpa_bwd(q, k, v, o, lse, dout, dq, dk, dv, cu_seqlens, B, Hq, Hkv, D, causal, scale, total_tokens,
                    max_seqlen, scratch, static_cast<size_t>(SDPA_STATIC_SCRATCH_BYTES), stream);
}

extern "C" int sdpa_bwd_profile_events(void* ev_main_start, void* ev_main_stop) {
    tl_ev_main_start = static_cast<cudaEvent_t>(ev_main_start);
    tl_ev_main_stop = static_cast<cudaEvent_t>(ev_main_stop);
    return SDPA_OK;
}

extern "C" size_t sdpa_host_staging_bytes(int B, int Hq, int Hkv, int D, int total_tokens, int max_seqlen) {
    const size_t ws = sdpa_bwd_workspace_bytes(B, Hq, Hkv, D, total_tokens, max_seqlen);
    if (ws == 0) return 0;
    const size_t T = static_cast<size_t>(total_tokens);
    const size_t qb = T * Hq * D * 2, kb = T * Hkv * D * 2, lb = T * Hq * 4;
    const size_t cb = align_up(static_cast<size_t>(B + 1) * 4, 256);
    // q, dout, o, dq + k, v, dk, dv + lse, cut into at most 8 chunks of 9 separately aligned pieces
    return 4 * qb + 4 * kb + lb + cb + align_up(ws, 256) + 8 * 9 * 256;
}

// Copy streams and events of sdpa_fwd_bwd_host, one set per (host thread, device), created on first use
// and kept for the life of the thread.
constexpr int kHostMaxChunks = 8;
struct HostPipe {
    bool ready = false;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_out = nullptr;
    cudaEvent_t ev_in[kHostMaxChunks] = {}, ev_cmp[kHostMaxChunks] = {};
};
static thread_local HostPipe tl_pipe[sdpa::kMaxDevices];

static int host_pipe(HostPipe** out) {
    int dev = -1;
    SDPA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= sdpa::kMaxDevices) return SDPA_ERR_ARCH;
    HostPipe& hp = tl_pipe[dev];
    if (!hp.ready) {
        SDPA_CUDA_TRY(cudaStreamCreateWithFlags(&hp.s_in, cudaStreamNonBlocking));
        SDPA_CUDA_TRY(cudaStreamCreateWithFlags(&hp.s_out, cudaStreamNonBlocking));
        SDPA_CUDA_TRY(cudaEventCreateWithFlags(&hp.ev_start, cudaEventDisableTiming));
        SDPA_CUDA_TRY(cudaEventCreateWithFlags(&hp.ev_out, cudaEventDisableTiming));
        for (int i = 0; i < kHostMaxChunks; ++i) {
            SDPA_CUDA_TRY(cudaEventCreateWithFlags(&hp.ev_in[i], cudaEventDisableTiming));
            SDPA_CUDA_TRY(cudaEventCreateWithFlags(&hp.ev_cmp[i], cudaEventDisableTiming));
        }
        hp.ready = true;
    }
    *out = &hp;
    return SDPA_OK;
}

// The step is cut into chunks of kv heads (with their query heads): heads are independent problems, so
// while chunk c computes on the caller's stream, chunk c+1 is copied in on one copy stream and chunk c-1
// is copied out on another.  PCIe is full duplex, so the step costs about max(copy in, copy out) instead
// of their sum.  Chunks are taken out of the host tensors with pitched copies ([T, H, D] rows, a head
// range per chunk) and live on the device as contiguous [T, Hc, D] tensors.
extern "C" int sdpa_fwd_bwd_host(const void* q, const void* k, const void* v, const void* dout, void* o, float* lse,
                                 void* dq, void* dk, void* dv, const int32_t* cu_seqlens, int B, int Hq, int Hkv,
                                 int D, int causal, float scale, int total_tokens, int max_seqlen, void* staging,
                                 size_t staging_bytes, void* stream) {
    int rc = check_common(cu_seqlens, B, Hq, Hkv, D, scale, total_tokens, max_seqlen);
    if (rc != SDPA_OK) return rc;
    if (total_tokens == 0 || max_seqlen == 0) return SDPA_OK;
    if (!q || !k || !v || !dout || !o || !lse || !dq || !dk || !dv) return SDPA_ERR_NULL;
    const size_t need = sdpa_host_staging_bytes(B, Hq, Hkv, D, total_tokens, max_seqlen);
    if (staging == nullptr || (reinterpret_cast<uintptr_t>(staging) & 255u) || staging_bytes < need)
        return SDPA_ERR_WORKSPACE;
    HostPipe* hp = nullptr;
    if ((rc = host_pipe(&hp)) != SDPA_OK) return rc;

    const size_t T = static_cast<size_t>(total_tokens);
    const int G = Hq / Hkv;
    const int n_chunks = Hkv < 4 ? Hkv : 4;
    const size_t row = static_cast<size_t>(D) * 2;  // bytes of one head row
    const size_t c_bytes = static_cast<size_t>(B + 1) * 4;
    uint8_t* base = static_cast<uint8_t*>(staging);
    size_t off = 0;
    auto take = [&](size_t bytes) { uint8_t* p = base + off; off += align_up(bytes, 256); return p; };
    uint8_t* d_cu = take(c_bytes);
    // the backward workspace is shared by the chunks (they run one after the other on the caller's stream)
    const size_t ws_bytes = sdpa_bwd_workspace_bytes(B, Hq, Hkv, D, total_tokens, max_seqlen);
    uint8_t* d_ws = take(ws_bytes);

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    SDPA_CUDA_TRY(cudaEventRecord(hp->ev_start, s));
    SDPA_CUDA_TRY(cudaStreamWaitEvent(hp->s_in, hp->ev_start, 0));
    SDPA_CUDA_TRY(cudaMemcpyAsync(d_cu, cu_seqlens, c_bytes, cudaMemcpyHostToDevice, hp->s_in));
    for (int c = 0; c < n_chunks; ++c) {
        const int g0 = static_cast<int>(static_cast<long long>(Hkv) * c / n_chunks);
        const int g1 = static_cast<int>(static_cast<long long>(Hkv) * (c + 1) / n_chunks);
        const int hk = g1 - g0, hq = hk * G, h0 = g0 * G;
        const size_t qw = hq * row, kw = hk * row;  // bytes per token of the chunk's q-like / k-like tensors
        uint8_t* d_q = take(T * qw); uint8_t* d_do = take(T * qw); uint8_t* d_o = take(T * qw); uint8_t* d_dq = take(T * qw);
        uint8_t* d_k = take(T * kw); uint8_t* d_v = take(T * kw); uint8_t* d_dk = take(T * kw); uint8_t* d_dv = take(T * kw);
        uint8_t* d_lse = take(T * hq * 4);
        if (off > staging_bytes) return SDPA_ERR_WORKSPACE;
        const size_t qp = static_cast<size_t>(Hq) * row, kp = static_cast<size_t>(Hkv) * row;  // host pitches
        const uint8_t* hq_src = static_cast<const uint8_t*>(q) + h0 * row;
        const uint8_t* hdo_src = static_cast<const uint8_t*>(dout) + h0 * row;
        const uint8_t* hk_src = static_cast<const uint8_t*>(k) + g0 * row;
        const uint8_t* hv_src = static_cast<const uint8_t*>(v) + g0 * row;
        SDPA_CUDA_TRY(cudaMemcpy2DAsync(d_q, qw, hq_src, qp, qw, T, cudaMemcpyHostToDevice, hp->s_in));
        SDPA_CUDA_TRY(cudaMemcpy2DAsync(d_k, kw, hk_src, kp, kw, T, cudaMemcpyHostToDevice, hp->s_in));
        SDPA_CUDA_TRY(cudaMemcpy2DAsync(d_v, kw, hv_src, kp, kw, T, cudaMemcpyHostToDevice, hp->s_in));
        SDPA_CUDA_TRY(cudaMemcpy2DAsync(d_do, qw, hdo_src, qp, qw, T, cudaMemcpyHostToDevice, hp->s_in));
        SDPA_CUDA_TRY(cudaEventRecord(hp->ev_in[c], hp->s_in));

        SDPA_CUDA_TRY(cudaStreamWaitEvent(s, hp->ev_in[c], 0));
        rc = sdpa_fwd(d_q, d_k, d_v, d_o, reinterpret_cast<float*>(d_lse), reinterpret_cast<const int32_t*>(d_cu), B, hq,
                      hk, D, causal, scale, total_tokens, max_seqlen, stream);
        if (rc != SDPA_OK) return rc;
        rc = sdpa_bwd(d_q, d_k, d_v, d_o, reinterpret_cast<const float*>(d_lse), d_do, d_dq, d_dk, d_dv,
                      reinterpret_cast<const int32_t*>(d_cu), B, hq, hk, D, causal, scale, total_tokens, max_seqlen,
                      d_ws, ws_bytes, stream);
        if (rc != SDPA_OK) return rc;
        SDPA_CUDA_TRY(cudaEventRecord(hp->ev_cmp[c], s));

        SDPA_CUDA_TRY(cudaStreamWaitEvent(hp->s_out, hp->ev_cmp[c], 0));
        uint8_t* ho = static_cast<uint8_t*>(o) + h0 * row;
        uint8_t* hdq = static_cast<uint8_t*>(dq) + h0 * row;
        uint8_t* hdk = static_cast<uint8_t*>(dk) + g0 * row;
        uint8_t* hdv = static_cast<uint8_t*>(dv) + g0 * row;
        SDPA_CUDA_TRY(cudaMemcpy2DAsync(ho, qp, d_o, qw, qw, T, cudaMemcpyDeviceToHost, hp->s_out));
        SDPA_CUDA_TRY(cudaMemcpyAsync(lse + static_cast<size_t>(h0) * T, d_lse, T * hq * 4, cudaMemcpyDeviceToHost, hp->s_out));
        SDPA_CUDA_TRY(cudaMemcpy2DAsync(hdq, qp, d_dq, qw, qw, T, cudaMemcpyDeviceToHost, hp->s_out));
        SDPA_CUDA_TRY(cudaMemcpy2DAsync(hdk, kp, d_dk, kw, kw, T, cudaMemcpyDeviceToHost, hp->s_out));
        SDPA_CUDA_TRY(cudaMemcpy2DAsync(hdv, kp, d_dv, kw, kw, T, cudaMemcpyDeviceToHost, hp->s_out));
    }
    // join: everything after this call on the caller's stream sees the finished host outputs
    SDPA_CUDA_TRY(cudaEventRecord(hp->ev_out, hp->s_out));
    SDPA_CUDA_TRY(cudaStreamWaitEvent(s, hp->ev_out, 0));
    return SDPA_OK;
}

// Tensor map over a row-major bf16 matrix [rows, cols]: dims {cols, rows}, box {64, box_rows}, 128B swizzle.
static int make_map_2d(CUtensorMap* map, const void* base, int rows, int cols, int box_rows) {
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * 2};
    const cuuint32_t box[2] = {64, static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                                estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        tl_last_cuda_error = static_cast<int>(r);
        return SDPA_ERR_CUDA;
    }
    return SDPA_OK;
}

extern "C" int gemm_bf16_nt(const void* a, const void* b, void* c, int M, int N, int K, void* stream) {
    if (M < 0 || N < 0 || K < 0) return SDPA_ERR_SHAPE;
    if ((K % 8) != 0 || (N % 8) != 0) return SDPA_ERR_SHAPE;  // 16-byte row pitches and 16-byte output vectors
    if (M == 0 || N == 0) return SDPA_OK;
    if (K == 0) return SDPA_ERR_SHAPE;
    if (!a || !b || !c) return SDPA_ERR_NULL;
    if (!aligned16(a) || !aligned16(b) || !aligned16(c)) return SDPA_ERR_ALIGN;
    DeviceState* st = nullptr;
    int rc = device_state(&st);
    if (rc != SDPA_OK) return rc;
    CUtensorMap ma, mb;
    if ((rc = make_map_2d(&ma, a, M, K, GemmCfg::BM)) != SDPA_OK) return rc;
    if ((rc = make_map_2d(&mb, b, N, K, GemmCfg::BN)) != SDPA_OK) return rc;
    GemmParams p;
    p.c = static_cast<__nv_bfloat16*>(c);
    p.status = st->status_ptr;
    p.M = M; p.N = N; p.K = K;
    const long long tiles = static_cast<long long>((M + GemmCfg::BM - 1) / GemmCfg::BM) * ((N + GemmCfg::BN - 1) / GemmCfg::BN);
    if (tiles > 2147483647ll) return SDPA_ERR_SHAPE;
    const unsigned grid = static_cast<unsigned>(tiles < st->num_sms ? tiles : st->num_sms);
    gemm_bf16_nt_kernel<<<grid, GemmCfg::kThreads, GemmCfg::kSmemBytes, static_cast<cudaStream_t>(stream)>>>(ma, mb, p);
    SDPA_CUDA_TRY(cudaGetLastError());
    return SDPA_OK;
}

// One warp waits on an mbarrier that nobody ever arrives at: exercises the bounded wait, the status
// word and the clean exit of a CTA without faulting or hanging the GPU.
__global__ void sdpa_selftest_wait_kernel(int* status, long long limit_cycles) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&bar, 1);
        fence_mbar_init();
    }
    __syncthreads();
    WaitCtl ctl{status, &abort_flag, limit_cycles};
    const bool ok = mbar_wait_warp(&bar, 0, ctl, 99);
    (void)ok;
}

extern "C" int sdpa_selftest_wait_timeout(long long limit_cycles, void* stream) {
    if (limit_cycles < 1 || limit_cycles > 4000000000ll) return SDPA_ERR_SHAPE;  // at most ~2 s
    DeviceState* st = nullptr;
    int rc = device_state(&st);
    if (rc != SDPA_OK) return rc;
    sdpa_selftest_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(st->status_ptr, limit_cycles);
    SDPA_CUDA_TRY(cudaGetLastError());
    return SDPA_OK;
}

extern "C" int sdpa_query_status(void* stream, int* site) {
    DeviceState* st = nullptr;
    int rc = device_state(&st);
    if (rc != SDPA_OK) return rc;
    SDPA_CUDA_TRY(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    int word = 0;
    SDPA_CUDA_TRY(cudaMemcpy(&word, st->status_ptr, sizeof(int), cudaMemcpyDeviceToHost));
    if (word != 0) SDPA_CUDA_TRY(cudaMemset(st->status_ptr, 0, sizeof(int)));
    if (site) *site = word >> 8;
    return word & 0xff;
}

extern "C" const char* sdpa_status_string(int code) {
    switch (code) {
        case SDPA_OK: return "ok";
        case SDPA_ERR_NULL: return "null pointer argument";
        case SDPA_ERR_ALIGN: return "pointer not 16-byte aligned";
        case SDPA_ERR_SHAPE: return "unsupported shape or scale";
        case SDPA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case SDPA_ERR_ARCH: return "device is not compute capability 10.x";
        case SDPA_ERR_CUDA: return "CUDA runtime or driver call failed";
        case SDPA_ERR_STATIC_SCRATCH:
            return "problem exceeds the built-in scratch (SDPA_STATIC_SCRATCH_BYTES); use sdpa_bwd with a workspace";
        case SDPA_STATUS_TIMEOUT: return "device-side wait timed out";
        case SDPA_STATUS_BAD_CU_SEQLENS: return "cu_seqlens inconsistent with total_tokens/max_seqlen";
        case SDPA_STATUS_INTERNAL: return "kernel launch precondition violated";
        default: return "unknown code";
    }
}

extern "C" int sdpa_last_cuda_error(void) { return tl_last_cuda_error; }

#ifdef SDPA_TRACE
extern "C" int sdpa_debug_trace(long long* host_out, int n) {
    return static_cast<int>(cudaMemcpyFromSymbol(host_out, sdpa::g_trace, sizeof(long long) * n));
}
#endif
