// based_prefill for the feature dimensions 8, 24 and 32 (bf16 io): the final recurrent state
// (Sec. 4.1, Eq. (3): S = sum_j phi(k_j) v_j^T, z = sum_j phi(k_j)) on the tensor cores.
//
//   S[f, :] (+)= sum_j phi_f(k_j) v_j        z[f] (+)= sum_j phi_f(k_j)
//
// in the state's own row order (row 0 constant, rows 1..d' linear, row 1 + d' + m d' + n the
// product k_m k_n).  One CTA per (block of 128 feature rows, head), 160 threads: the four row
// warps own one feature row (= accumulator lane) each, warp 4 (converged, one elected lane) issues TMA loads and
// MMAs.  Per step of 64 tokens the row threads transpose the k tile ([token][m] -> [m][token]),
// form their row of the A operand, [128 features][64 tokens] in the K-major SWIZZLE_128B layout,
// as packed bf16 products k_m k_n (eight tokens per instruction), and one MMA burst adds
// A x [V_j | 1] to the fp32 accumulator in tensor memory ([128 features][d_v + 16]; the ones
// block makes column d_v the row sum z).  The feature scales 1/d'^(1/4) and 1/(sqrt 2 sqrt d')
// multiply the fp32 sums at the end, so the operand carries one rounding (of the product) only.
// The A operand is double-buffered and the k / v tiles come through a ring of stages, so the
// loads, the row threads and the tensor pipe overlap.
#include <cuda_bf16.h>
#include <math.h>

#include <mutex>

#include "common.cuh"
#include "sm100.cuh"

namespace based {
using namespace sm100;

// [BH][L][width] bf16 tensor map with a [1][box_rows][box_w] box (defined with the backward kernels)
bool make_rows_map_bf16(CUtensorMap* m, const void* base, int BH, int L, int width, int box_w, int box_rows,
                        CUtensorMapSwizzle sw);

namespace {
constexpr int kFB = 128;           // feature rows per CTA (accumulator lanes)
constexpr int kTB = 64;            // tokens per step (K extent of one MMA burst)
constexpr int kThreadsS = 160;
constexpr int kKT = 72;            // row length of the transposed k tile (64 tokens + padding)
constexpr int kNA = 2;             // buffers of the A operand
constexpr int kRowOne = 32, kRowZero = 33;   // extra rows of the transposed tile: token-valid ones, zeros

template <int DV> struct SCfg {
    static constexpr int kVB = (DV + 63) / 64;                 // 64-column blocks of the v tile (112 -> 2)
    static constexpr int kNS = DV == 64 ? 4 : 3;               // load stages
    static constexpr uint32_t kVBytes = kVB * kTB * 128;       // [64 tokens][64 * kVB] bf16, SWIZZLE_128B blocks
    static constexpr uint32_t kKBytes = kTB * 64;              // [64 tokens][32] bf16, 64-byte rows, SWIZZLE_64B
    static constexpr uint32_t kStage = kVBytes + kKBytes;
    static constexpr uint32_t kABytes = kFB * 128;             // [128 features][64 tokens] bf16
    static constexpr uint32_t offA = kNS * kStage;
    static constexpr uint32_t offOnes = offA + kNA * kABytes;    // [16][64] bf16 ones (B operand of the row sums)
    static constexpr uint32_t offKT = offOnes + 2048;          // two transposed k tiles [34][kKT] bf16
    static constexpr uint32_t kKTBytes = 34 * kKT * 2;
    static constexpr uint32_t offMisc = offKT + 2 * kKTBytes + 64;
    static constexpr uint32_t kSmem = ((offMisc + 1023) / 1024) * 1024 + 256 + 1024;
    static constexpr uint32_t kCols = DV == 64 ? 128 : 256;    // accumulator: d_v + 16 columns
    static constexpr uint32_t colZ = 64 * kVB;
};
enum { sFull0 = 0, sAlu0 = 8, sMma0 = 12, sFinal = 16, sNum = 17 };      // up to 8 load stages, 4 A buffers

struct SParams {
    float* kv;                     // [BH, D, dvw]
    float* z;                      // [BH, D]
    unsigned int* err;
    int L, df, D, dvw, cont;
    float lin, quad;
};

// AND of a predicate over the 128 row threads (named barrier 2); also a barrier for their shared-memory traffic
__device__ __forceinline__ bool rows_and(bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 2, 128, p;\n\t"
        "selp.b32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred)
        : "memory");
    return r != 0;
}
}  // namespace

template <int DV>
__global__ void __launch_bounds__(kThreadsS, 1)
    generic_state_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                            const SParams p) {
    using C = SCfg<DV>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + ((C::offMisc + 1023) / 1024) * 1024);
    uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(bars + sNum);
    volatile uint32_t* abort_flag = tmem_base_s + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int head = blockIdx.y;
    const int f0 = blockIdx.x * kFB;
    const int nit = (p.L + kTB - 1) / kTB;

    if (tid == 0) {
        for (int s = 0; s < C::kNS; ++s) mbar_init(&bars[sFull0 + s], 1);
        for (int b = 0; b < kNA; ++b) { mbar_init(&bars[sAlu0 + b], 128); mbar_init(&bars[sMma0 + b], 1); }
        mbar_init(&bars[sFinal], 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    // constants in shared memory: the ones block, the zero rows of both transposed tiles
    {
        __nv_bfloat16* ones = reinterpret_cast<__nv_bfloat16*>(smem + C::offOnes);
        for (int i = tid; i < 1024; i += kThreadsS) ones[i] = __float2bfloat16(1.0f);
        for (int i = tid; i < 2 * kKT; i += kThreadsS) {
            __nv_bfloat16* kt = reinterpret_cast<__nv_bfloat16*>(smem + C::offKT + (i / kKT) * C::kKTBytes);
            kt[kRowZero * kKT + (i % kKT)] = __float2bfloat16(0.0f);
        }
    }
    fence_proxy_async_smem();
    if (warp == 4) { tmem_alloc(tmem_base_s, C::kCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = *tmem_base_s;
    bool ok = true;

    if (warp == 4) {
        {
            // the whole warp runs this block; one elected lane issues the MMAs, commits and loads (see mma_ss_w)
            const uint32_t lead = elect_one();
            constexpr uint64_t dA = make_smem_desc_base(16, 1024, kSwizzle128B);              // K-major, one 64-token block
            constexpr uint64_t dV = make_smem_desc_base(kTB * 128, 1024, kSwizzle128B);       // MN-major, 64-column blocks
            constexpr uint32_t iV = make_idesc_bf16(128, 64 * C::kVB, 0, 1);
            constexpr uint32_t iZ = make_idesc_bf16(128, 16, 0, 0);
            const uint32_t aOnes = smem_u32(smem + C::offOnes);
            auto load = [&](int it) {
                if (!lead) return;
                const int s = it % C::kNS;
                uint8_t* st = smem + s * C::kStage;
                mbar_arrive_expect_tx(&bars[sFull0 + s], C::kStage);
#pragma unroll
                for (int b = 0; b < C::kVB; ++b)
                    tma_load_3d(st + b * (kTB * 128), &tm_v, &bars[sFull0 + s], b * 64, it * kTB, head);
                tma_load_3d(st + C::kVBytes, &tm_k, &bars[sFull0 + s], 0, it * kTB, head);
            };
            for (int it = 0; it < C::kNS && it < nit; ++it) load(it);
            for (int it = 0; it < nit && ok; ++it) {
                const int b = it % kNA, s = it % C::kNS;
                ok = mbar_wait(&bars[sFull0 + s], (it / C::kNS) & 1, abort_flag);
                if (!ok) break;
                ok = mbar_wait(&bars[sAlu0 + b], (it / kNA) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t aA = smem_u32(smem + C::offA + b * C::kABytes), aV = smem_u32(smem + s * C::kStage);
#pragma unroll
                for (int kk = 0; kk < kTB / 16; ++kk) {
                    if (it == 0 && kk == 0) {
                        mma_ss_w<false>(lead, tb, desc_lo(dA) + ((aA + kk * 32) >> 4), desc_hi(dA),
                                         desc_lo(dV) + ((aV + kk * 2048) >> 4), desc_hi(dV), iV);
                        mma_ss_w<false>(lead, tb + C::colZ, desc_lo(dA) + ((aA + kk * 32) >> 4), desc_hi(dA),
                                         desc_lo(dA) + ((aOnes + kk * 32) >> 4), desc_hi(dA), iZ);
                    } else {
                        mma_ss_w<true>(lead, tb, desc_lo(dA) + ((aA + kk * 32) >> 4), desc_hi(dA),
                                        desc_lo(dV) + ((aV + kk * 2048) >> 4), desc_hi(dV), iV);
                        mma_ss_w<true>(lead, tb + C::colZ, desc_lo(dA) + ((aA + kk * 32) >> 4), desc_hi(dA),
                                        desc_lo(dA) + ((aOnes + kk * 32) >> 4), desc_hi(dA), iZ);
                    }
                }
                mma_commit_w(lead, &bars[sMma0 + b]);
                // the previous step's products are done long since: its stage takes the load kNS steps ahead
                if (it >= 1 && it - 1 + C::kNS < nit) {
                    ok = mbar_wait(&bars[sMma0 + (it - 1) % kNA], ((it - 1) / kNA) & 1, abort_flag);
                    if (!ok) break;
                    load(it - 1 + C::kNS);
                }
            }
            if (ok) mma_commit_w(lead, &bars[sFinal]);
        }
    } else {
        // ===================================================================== row threads
        const int t = tid;                                   // accumulator lane
        const int f = f0 + t;                                // state row
        // the row's factors as rows of the transposed k tile: k_m k_n, k_m x 1, 1 x 1, or 0 past the last row
        int m = kRowZero, n = kRowZero;
        float scale = 0.f;
        if (f == 0) { m = kRowOne; n = kRowOne; scale = 1.0f; }
        else if (f <= p.df) { m = f - 1; n = kRowOne; scale = p.lin; }
        else if (f < p.D) { m = (f - 1 - p.df) / p.df; n = (f - 1 - p.df) % p.df; scale = p.quad; }
        uint8_t* a_row0 = smem + C::offA + t * 128;
        for (int it = 0; it < nit && ok; ++it) {
            const int b = it % kNA, s = it % C::kNS;
            ok = rows_and(mbar_wait(&bars[sFull0 + s], (it / C::kNS) & 1, abort_flag));
            if (!ok) break;
            // transpose the k tile ([token][m], 64-byte rows, SWIZZLE_64B): warp w moves the 16-byte pieces
            // w / 2 and w / 2 + 2 of tokens 32 (w % 2) + lane, so a warp's loads hit distinct banks and its
            // 2-byte stores fill consecutive words of one transposed row
            __nv_bfloat16* kt = reinterpret_cast<__nv_bfloat16*>(smem + C::offKT + (it & 1) * C::kKTBytes);
            {
                const int j = lane + 32 * (warp & 1);
                const uint8_t* krow = smem + s * C::kStage + C::kVBytes + j * 64;
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    const int c = (warp >> 1) + 2 * cc;
                    const uint4 u = *reinterpret_cast<const uint4*>(krow + ((c ^ ((j >> 1) & 3)) << 4));
                    const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&u);
#pragma unroll
                    for (int i = 0; i < 8; ++i) kt[(c * 8 + i) * kKT + j] = e[i];
                }
                if (t < kTB) kt[kRowOne * kKT + t] = __float2bfloat16(it * kTB + t < p.L ? 1.0f : 0.0f);
            }
            // the A buffer is free once the products of kNA steps ago are done; the barrier also publishes the transpose
            ok = rows_and(it < kNA || mbar_wait(&bars[sMma0 + b], ((it / kNA) - 1) & 1, abort_flag));
            if (!ok) break;
            const uint4* rm = reinterpret_cast<const uint4*>(kt + m * kKT);
            const uint4* rn = reinterpret_cast<const uint4*>(kt + n * kKT);
            uint8_t* a_row = a_row0 + b * C::kABytes;
            uint4 xm[kTB / 8], xn[kTB / 8];                  // all sixteen loads in flight before the first product
#pragma unroll
            for (int c = 0; c < kTB / 8; ++c) { xm[c] = rm[c]; xn[c] = rn[c]; }
#pragma unroll
            for (int c = 0; c < kTB / 8; ++c) {
                uint4 pr;
                const __nv_bfloat162* hm = reinterpret_cast<const __nv_bfloat162*>(&xm[c]);
                const __nv_bfloat162* hn = reinterpret_cast<const __nv_bfloat162*>(&xn[c]);
                __nv_bfloat162* hp = reinterpret_cast<__nv_bfloat162*>(&pr);
#pragma unroll
                for (int i = 0; i < 4; ++i) hp[i] = __hmul2(hm[i], hn[i]);
                *reinterpret_cast<uint4*>(a_row + ((c ^ (t & 7)) << 4)) = pr;
            }
            fence_proxy_async_smem();
            mbar_arrive(&bars[sAlu0 + b]);
        }
        ok = rows_and(ok && mbar_wait(&bars[sFinal], 0, abort_flag));
        tc_fence_after();
        if (ok) {                                            // uniform over the row threads
            const uint32_t lane_base = (uint32_t)warp * 32u;
            const bool store = f < p.D;
            const size_t row = (size_t)head * p.D + (store ? f : 0);
            float* dst = p.kv + row * p.dvw;
            for (int c = 0; c < p.dvw / 16; ++c) {           // p.dvw is uniform: the loads stay warp-collective
                uint32_t r[16];
                tmem_ld16(tmem_addr(tb, lane_base, c * 16), r);
                tmem_wait_ld();
                if (store) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float4 o = make_float4(__uint_as_float(r[4 * i]) * scale, __uint_as_float(r[4 * i + 1]) * scale,
                                               __uint_as_float(r[4 * i + 2]) * scale, __uint_as_float(r[4 * i + 3]) * scale);
                        float4* d4 = reinterpret_cast<float4*>(dst + c * 16 + 4 * i);
                        if (p.cont) {
                            const float4 old = *d4;
                            o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                        }
                        *d4 = o;
                    }
                }
            }
            uint32_t zr;
            tmem_ld1(tmem_addr(tb, lane_base, C::colZ), zr);
            tmem_wait_ld();
            if (store) p.z[row] = __uint_as_float(zr) * scale + (p.cont ? p.z[row] : 0.f);
        }
    }
    if (!ok && lane == 0) atomicOr(p.err, 1u);
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);     // loads still in flight get time to land
    }
    __syncthreads();
    if (warp == 4) tmem_dealloc(tb, C::kCols);
}

namespace {
template <int DV>
based_status launch_state_dv(const void* k, const void* v, float* kv, float* z, int BH, int L, int df, int dvw,
                             int cont, cudaStream_t stream) {
    using C = SCfg<DV>;
    CUtensorMap tk, tv;
    if (!make_rows_map_bf16(&tk, k, BH, L, df, 32, kTB, CU_TENSOR_MAP_SWIZZLE_64B) ||
        !make_rows_map_bf16(&tv, v, BH, L, dvw, 64, kTB, CU_TENSOR_MAP_SWIZZLE_128B))
        return BASED_ERR_CUDA;
    SParams p{};
    if (error_word_ptr(&p.err) != BASED_OK) return BASED_ERR_CUDA;
    p.kv = kv;
    p.z = z;
    p.L = L;
    p.df = df;
    p.D = 1 + df + df * df;
    p.dvw = dvw;
    p.cont = cont;
    const float rd = sqrtf((float)df);
    p.lin = 1.0f / sqrtf(rd);
    p.quad = 1.0f / (1.41421356237309505f * rd);
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BASED_ERR_CUDA;
    {
        std::lock_guard<std::mutex> lock(setup_mutex());
        if (!configured[dev]) {
            if (cudaFuncSetAttribute(generic_state_tc_kernel<DV>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)C::kSmem) != cudaSuccess)
                return BASED_ERR_CUDA;
            configured[dev] = true;
        }
    }
    generic_state_tc_kernel<DV><<<dim3((p.D + kFB - 1) / kFB, BH), kThreadsS, C::kSmem, stream>>>(tk, tv, p);
    note_launch();
    return check_launch("generic_state_tc_kernel");
}
}  // namespace

based_status launch_state_generic_tc(const void* k, const void* v, float* kv, float* z, int BH, int L, int d_feat,
                                     int d_v, int cont, cudaStream_t stream) {
    if (d_v == 64) return launch_state_dv<64>(k, v, kv, z, BH, L, d_feat, 64, cont, stream);
    return launch_state_dv<128>(k, v, kv, z, BH, L, d_feat, d_v, cont, stream);        // 112 or 128
}

}  // namespace based
