// swa_forward, SIMT path: exact causal softmax attention inside a sliding window
// (Eq. (1) of Sec. 2 with the key set {i-w+1..i} of Sec. 4.2), fp32 arithmetic.
//
// One CTA handles 64 consecutive queries of one head; the keys and values they can
// see (at most 64 + window - 1 rows) are staged once in shared memory as fp32, so
// every k, v row is read from HBM once per CTA.  A warp walks its 8 queries: lane l
// scores window slots l, l+32, ... (key i - slot), the warp reduces max and sum with
// shuffles, and each lane then accumulates two output columns over the window.
#include <math.h>

#include "common.cuh"

namespace based {

namespace {
constexpr int kQT = 64;          // queries per CTA
constexpr int kHD = 64;          // head dimension
constexpr int kMaxWin = 128;
constexpr int kKeyRows = kQT + kMaxWin;   // >= 64 + 127
constexpr int kKStride = kHD + 1;         // padded row: lanes reading different keys hit different banks
constexpr size_t kSmemBytes = sizeof(float) * (kKeyRows * kKStride + kKeyRows * kHD + kQT * kHD + 8 * kMaxWin);
}  // namespace

template <typename T>
__global__ void __launch_bounds__(256) swa_simt_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                       const T* __restrict__ v, T* __restrict__ out, int L,
                                                       int window, float scale) {
    extern __shared__ __align__(16) float smem[];
    float* sK = smem;                               // [kKeyRows][kKStride]
    float* sV = sK + kKeyRows * kKStride;           // [kKeyRows][kHD]
    float* sQ = sV + kKeyRows * kHD;                // [kQT][kHD]
    float* sP = sQ + kQT * kHD;                     // [8][kMaxWin]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const size_t head = blockIdx.y;
    const int i0 = blockIdx.x * kQT;
    const int nq = min(kQT, L - i0);
    const int ks = max(0, i0 - (window - 1));       // first key any query of this tile sees
    const int nk = i0 + nq - ks;

    const T* qh = q + (head * L + i0) * kHD;
    const T* kh = k + (head * L + ks) * kHD;
    const T* vh = v + (head * L + ks) * kHD;
    for (int i = tid; i < nq * kHD; i += 256) sQ[i] = to_f32(qh[i]);
    for (int i = tid; i < nk * kHD; i += 256) {
        sK[(i / kHD) * kKStride + (i % kHD)] = to_f32(kh[i]);
        sV[i] = to_f32(vh[i]);
    }
    __syncthreads();

    float* p = sP + warp * kMaxWin;
    for (int iq = warp; iq < nq; iq += 8) {
        const int i = i0 + iq;
        const int nwin = min(window, i + 1);        // keys i, i-1, ..., i-nwin+1
        float sc[kMaxWin / 32];
        float mx = -INFINITY;
#pragma unroll
        for (int u = 0; u < kMaxWin / 32; ++u) {
            const int s = lane + 32 * u;
            sc[u] = -INFINITY;
            if (s < nwin) {
                const float* kr = sK + (i - s - ks) * kKStride;
                const float* qr = sQ + iq * kHD;
                float a = 0.f;
#pragma unroll 16
                for (int m = 0; m < kHD; ++m) a = fmaf(qr[m], kr[m], a);
                sc[u] = a * scale;
                mx = fmaxf(mx, sc[u]);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float sum = 0.f;
#pragma unroll
        for (int u = 0; u < kMaxWin / 32; ++u) {
            const int s = lane + 32 * u;
            if (s < nwin) {
                const float e = expf(sc[u] - mx);
                p[s] = e;
                sum += e;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        __syncwarp();
        float a0 = 0.f, a1 = 0.f;
        for (int s = 0; s < nwin; ++s) {
            const float* vr = sV + (i - s - ks) * kHD;
            a0 = fmaf(p[s], vr[lane], a0);
            a1 = fmaf(p[s], vr[lane + 32], a1);
        }
        T* o = out + (head * L + i) * kHD;
        o[lane] = from_f32<T>(a0 / sum);
        o[lane + 32] = from_f32<T>(a1 / sum);
        __syncwarp();
    }
}

template <typename T>
static based_status launch_t(const void* q, const void* k, const void* v, void* out, int BH, int L, int window,
                             float scale, cudaStream_t stream) {
    // per-device attribute; setting it on every call keeps multi-device processes correct
    if (cudaFuncSetAttribute(swa_simt_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) !=
        cudaSuccess)
        return BASED_ERR_CUDA;
    dim3 grid((L + kQT - 1) / kQT, BH);
    swa_simt_kernel<T><<<grid, 256, kSmemBytes, stream>>>(static_cast<const T*>(q), static_cast<const T*>(k),
                                                          static_cast<const T*>(v), static_cast<T*>(out), L, window,
                                                          scale);
    note_launch();
    return check_launch("swa_simt_kernel");
}

based_status launch_swa_simt(const void* q, const void* k, const void* v, void* out, int BH, int L, int window,
                             float scale, based_dtype io, cudaStream_t stream) {
    return io == BASED_F32 ? launch_t<float>(q, k, v, out, BH, L, window, scale, stream)
                           : launch_t<__nv_bfloat16>(q, k, v, out, BH, L, window, scale, stream);
}

}  // namespace based
