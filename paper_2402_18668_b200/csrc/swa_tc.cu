// swa_forward, bf16 tensor-core path (tcgen05 + TMEM + TMA): exact causal softmax
// attention in a sliding window (Eq. (1) of Sec. 2 with the key set {i-w+1..i} of
// Sec. 4.2), head dimension 64, window <= 64.
//
// One CTA per tile of 128 consecutive queries of one head.  The 192 keys the tile can see
// (64 before its first query, then its own 128) are loaded once; per tile
//   S[128,192] = Q K^T          4 MMAs (K = 64), fp32 in TMEM
//   softmax    one thread per query row reads the 96 columns its warp's rows can touch,
//              masks to its own window, exp2 with the scale folded in, writes P (bf16) back
//              into TMEM over the scores
//   O[128,64]  = P V            12 MMAs with P read from TMEM
//   out        O / rowsum -> bf16 -> swizzled shared tile -> TMA store.
// The kernel is bound by HBM (512 B per token and head against ~50 k flop): two CTAs are
// resident per SM so one tile's loads overlap the other's arithmetic.
#include <cuda_bf16.h>

#include "common.cuh"
#include "sm100.cuh"

namespace based {

using namespace sm100;

namespace {

constexpr int kQT = 128;                 // queries per tile
constexpr int kPad = 64;                 // keys loaded before the tile's first query (>= window - 1)
constexpr int kKeys = kQT + kPad;        // 192
constexpr int kHD = 64;
constexpr int kThreads = 160;            // 4 softmax warps + 1 producer/MMA warp
constexpr uint32_t kQBytes = kQT * kHD * 2;      // 16 KB
constexpr uint32_t kKVBytes = kKeys * kHD * 2;   // 24 KB
constexpr uint32_t offQ = 0, offK = kQBytes, offV = kQBytes + kKVBytes, offBars = kQBytes + 2 * kKVBytes;
constexpr uint32_t kSmemBytes = 100 * 1024;   // > 1/3 of an SM: at most two CTAs (2 x 256 TMEM columns) per SM
static_assert(offBars + 128 + 1024 <= kSmemBytes, "shared memory layout");
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t colS = 0, colO = 128;         // P overwrites columns [0, 96) of S; O uses dead S columns

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

struct SwaParams {
    unsigned int* err;
    int L;
    int window;
    float scale_log2e;      // softmax scale * log2(e)
};

}  // namespace

__global__ void __launch_bounds__(kThreads, 2)
    swa_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                  const SwaParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + offBars);      // 0 loads, 1 scores, 2 P, 3 O
    uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(bars + 4);
    volatile uint32_t* abort_flag = tmem_base_s + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int head = blockIdx.y;
    const int i0 = blockIdx.x * kQT;

    if (tid == 0) {
        mbar_init(&bars[0], 1); mbar_init(&bars[1], 1); mbar_init(&bars[2], 128); mbar_init(&bars[3], 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 4) { tmem_alloc(tmem_base_s, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = *tmem_base_s;
    bool ok = true;

    if (warp == 4) {
        if (lane == 0) {
            // ---- loads: Q tile, and K, V rows i0-64 .. i0+127 (rows before the sequence start read as zero)
            mbar_arrive_expect_tx(&bars[0], kQBytes + 2 * kKVBytes);
            tma_load_3d(smem + offQ, &tm_q, &bars[0], 0, i0, head);
            tma_load_3d(smem + offK, &tm_k, &bars[0], 0, i0 - kPad, head);
            tma_load_3d(smem + offV, &tm_v, &bars[0], 0, i0 - kPad, head);
            constexpr uint64_t dK = make_smem_desc_base(16, 1024, kSwizzle128B);   // K-major, 128-byte rows
            constexpr uint64_t dVmn = make_smem_desc_base(16, 1024, kSwizzle128B); // MN-major, one 64-column block
            constexpr uint32_t iS = make_idesc_bf16(kQT, kKeys, 0, 0);
            constexpr uint32_t iO = make_idesc_bf16(kQT, kHD, 0, 1);
            const uint32_t lQ = desc_lo(dK) + (smem_u32(smem + offQ) >> 4);
            const uint32_t lK = desc_lo(dK) + (smem_u32(smem + offK) >> 4);
            const uint32_t lV = desc_lo(dVmn) + (smem_u32(smem + offV) >> 4);
            ok = mbar_wait(&bars[0], 0, abort_flag);
            if (ok) {
                tc_fence_after();
                mma_ss_lh<false>(tb + colS, lQ, desc_hi(dK), lK, desc_hi(dK), iS);
#pragma unroll
                for (int k = 1; k < kHD / 16; ++k)
                    mma_ss_lh<true>(tb + colS, lQ + k * 2, desc_hi(dK), lK + k * 2, desc_hi(dK), iS);
                mma_commit(&bars[1]);
                ok = mbar_wait(&bars[2], 0, abort_flag);
            }
            if (ok) {
                tc_fence_after();
                mma_ts_lh<false>(tb + colO, tb + colS, lV, desc_hi(dVmn), iO);
#pragma unroll
                for (int k = 1; k < kKeys / 16; ++k)
                    mma_ts_lh<true>(tb + colO, tb + colS + k * 8, lV + k * (2048 >> 4), desc_hi(dVmn), iO);
                mma_commit(&bars[3]);
            }
        }
    } else {
        // ---- softmax: thread = query row r of the tile, TMEM lane r
        const int r = tid;
        const uint32_t lane_base = (uint32_t)warp * 32u;
        const int c0 = warp * 32;                    // first score column this warp reads (96 columns from here)
        // visible columns of this row inside the 96-column batch: keys i-w+1 .. i, and key >= 0
        const int jhi = lane + kPad;
        int jlo = lane + kPad + 1 - p.window;
        jlo = max(jlo, kPad - i0 - c0);              // key index i0 - 64 + c0 + j must not be negative
        auto mask_word = [&](int base) -> uint32_t {
            const int a = max(jlo - base, 0), b = min(jhi - base, 31);
            if (a > b) return 0u;
            return (b - a == 31) ? 0xffffffffu : (((1u << (b - a + 1)) - 1u) << a);
        };
        const uint32_t mk[3] = {mask_word(0), mask_word(32), mask_word(64)};

        ok = mbar_wait(&bars[1], 0, abort_flag);
        float inv_l = 0.f;
        if (ok) {
            tc_fence_after();
            uint32_t s[96];
            {
                uint32_t t0[32], t1[32], t2[32];
                tmem_ld32(tmem_addr(tb, lane_base, colS + c0), t0);
                tmem_ld32(tmem_addr(tb, lane_base, colS + c0 + 32), t1);
                tmem_ld32(tmem_addr(tb, lane_base, colS + c0 + 64), t2);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) { s[i] = t0[i]; s[32 + i] = t1[i]; s[64 + i] = t2[i]; }
            }
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < 96; ++j) {
                const bool v = (mk[j >> 5] >> (j & 31)) & 1u;
                const float x = v ? __uint_as_float(s[j]) : -INFINITY;
                s[j] = __float_as_uint(x);
                mx = fmaxf(mx, x);
            }
            const float mc = mx * p.scale_log2e;     // every row sees at least its own key, so mx is finite
            float l = 0.f;
            uint32_t pk[48];
#pragma unroll
            for (int j = 0; j < 48; ++j) {
                const float e0 = ex2(fmaf(__uint_as_float(s[2 * j]), p.scale_log2e, -mc));
                const float e1 = ex2(fmaf(__uint_as_float(s[2 * j + 1]), p.scale_log2e, -mc));
                l += e0 + e1;
                pk[j] = pack2(e0, e1);
            }
            inv_l = 1.0f / l;
            // P row: 192 keys = 96 packed columns; this warp's batch sits at packed columns [16w, 16w+48)
            uint32_t zero[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) zero[i] = 0u;
#pragma unroll
            for (int g = 0; g < 6; ++g)
                if (g < warp || g > warp + 2) tmem_st16(tmem_addr(tb, lane_base, colS + g * 16), zero);
            {
                uint32_t d0[16], d1[16], d2[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) { d0[i] = pk[i]; d1[i] = pk[16 + i]; d2[i] = pk[32 + i]; }
                tmem_st16(tmem_addr(tb, lane_base, colS + warp * 16), d0);
                tmem_st16(tmem_addr(tb, lane_base, colS + warp * 16 + 16), d1);
                tmem_st16(tmem_addr(tb, lane_base, colS + warp * 16 + 32), d2);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&bars[2]);
            ok = mbar_wait(&bars[3], 0, abort_flag);
        }
        if (ok) {
            tc_fence_after();
            uint32_t o0[32], o1[32];
            tmem_ld32(tmem_addr(tb, lane_base, colO), o0);
            tmem_ld32(tmem_addr(tb, lane_base, colO + 32), o1);
            tmem_wait_ld();
            // the Q tile is dead (its MMAs completed before the scores were signalled): stage the output there
            uint8_t* orow = smem + offQ + (r >> 3) * 1024 + (r & 7) * 128;
            const uint32_t sw = r & 7;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint4 v4;
                v4.x = pack2(__uint_as_float(o0[8 * j + 0]) * inv_l, __uint_as_float(o0[8 * j + 1]) * inv_l);
                v4.y = pack2(__uint_as_float(o0[8 * j + 2]) * inv_l, __uint_as_float(o0[8 * j + 3]) * inv_l);
                v4.z = pack2(__uint_as_float(o0[8 * j + 4]) * inv_l, __uint_as_float(o0[8 * j + 5]) * inv_l);
                v4.w = pack2(__uint_as_float(o0[8 * j + 6]) * inv_l, __uint_as_float(o0[8 * j + 7]) * inv_l);
                *reinterpret_cast<uint4*>(orow + ((j ^ sw) << 4)) = v4;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint4 v4;
                v4.x = pack2(__uint_as_float(o1[8 * j + 0]) * inv_l, __uint_as_float(o1[8 * j + 1]) * inv_l);
                v4.y = pack2(__uint_as_float(o1[8 * j + 2]) * inv_l, __uint_as_float(o1[8 * j + 3]) * inv_l);
                v4.z = pack2(__uint_as_float(o1[8 * j + 4]) * inv_l, __uint_as_float(o1[8 * j + 5]) * inv_l);
                v4.w = pack2(__uint_as_float(o1[8 * j + 6]) * inv_l, __uint_as_float(o1[8 * j + 7]) * inv_l);
                *reinterpret_cast<uint4*>(orow + (((4 + j) ^ sw) << 4)) = v4;
            }
            fence_proxy_async_smem();
        }
    }

    if (!ok && lane == 0) atomicOr(p.err, 1u);
    tc_fence_before();
    __syncthreads();
    if (!*abort_flag && tid == 0) {
        tma_store_3d(&tm_o, smem + offQ, 0, i0, head);      // rows past the sequence end are clipped
        tma_store_commit();
        tma_store_wait_read<0>();                           // shared memory must outlive the store's reads
    }
    if (*abort_flag) {
        for (int it = 0; it < 200; ++it) __nanosleep(1000);
    }
    __syncthreads();
    if (warp == 4) tmem_dealloc(tb, kTmemCols);
}

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool make_map(CUtensorMap* m, const void* base, int BH, int L, int box_rows) {
    static EncodeTiledFn enc = nullptr;
    if (!enc) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return false;
        enc = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    cuuint64_t dims[3] = {(cuuint64_t)kHD, (cuuint64_t)L, (cuuint64_t)BH};
    cuuint64_t strides[2] = {(cuuint64_t)kHD * 2, (cuuint64_t)L * kHD * 2};
    cuuint32_t box[3] = {(cuuint32_t)kHD, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool swa_tc_supported(int window) { return window >= 1 && window <= kPad; }

based_status launch_swa_tc(const void* q, const void* k, const void* v, void* out, int BH, int L, int window,
                           float scale, cudaStream_t stream) {
    CUtensorMap tq, tk, tv, to;
    if (!make_map(&tq, q, BH, L, kQT) || !make_map(&tk, k, BH, L, kKeys) || !make_map(&tv, v, BH, L, kKeys) ||
        !make_map(&to, out, BH, L, kQT))
        return BASED_ERR_CUDA;
    SwaParams p;
    if (error_word_ptr(&p.err) != BASED_OK) return BASED_ERR_CUDA;
    p.L = L;
    p.window = window;
    p.scale_log2e = scale * 1.4426950408889634f;
    if (cudaFuncSetAttribute(swa_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) !=
        cudaSuccess)
        return BASED_ERR_CUDA;
    dim3 grid((L + kQT - 1) / kQT, BH);
    swa_tc_kernel<<<grid, kThreads, kSmemBytes, stream>>>(tq, tk, tv, to, p);
    note_launch();
    return check_launch("swa_tc_kernel");
}

}  // namespace based
