// swa_decode_step: one generation step of the sliding-window softmax mixer on a rolling cache
// of the last `window` keys and values (the PyTorch sliding-window listing and Algorithm 3 of
// App. B.2, here with the cache update included and for any position of the ring).
//
// One CTA of 128 threads per (b, h).  All loads are issued up front and kept packed (as loaded)
// in registers: thread j holds cached key j (one row per thread, 128-bit loads) and, as one of 8
// threads per row in 16 row groups, its share of the cached values; the new k, v are written into
// slot pos % window; then scores, block-wide max and sum, and the weighted sum run from registers.
// The step reads 2 * window * 64 elements per head once: it is bound by HBM bandwidth and, at
// small batch, by launch latency.
#include <math.h>

#include "common.cuh"

namespace based {

namespace {
constexpr int kHD = 64;
constexpr int kMaxWin = 128;

template <typename T> struct Raw8;   // 8 consecutive elements as loaded (converted to fp32 only when used)
template <> struct Raw8<__nv_bfloat16> {
    uint4 u;
    __device__ __forceinline__ void load(const __nv_bfloat16* p) { u = *reinterpret_cast<const uint4*>(p); }
    __device__ __forceinline__ void get(float (&x)[8]) const {
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __bfloat1622float2(h[i]);
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
        }
    }
};
template <> struct Raw8<float> {
    float4 a, b;
    __device__ __forceinline__ void load(const float* p) {
        a = *reinterpret_cast<const float4*>(p);
        b = *reinterpret_cast<const float4*>(p + 4);
    }
    __device__ __forceinline__ void get(float (&x)[8]) const {
        x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
    }
};

}  // namespace

template <typename T, int VROWS>     // VROWS: value rows per thread = ceil(window / 16)
__global__ void __launch_bounds__(128, (sizeof(T) == 2 && VROWS <= 4) ? 8 : 4)
swa_decode_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v, T* __restrict__ kc,
                  T* __restrict__ vc, T* __restrict__ out, int window, int pos, float scale) {
    __shared__ float s_q[kHD];
    __shared__ float s_p[kMaxWin];
    __shared__ float s_red[8];
    __shared__ __align__(16) float s_acc[16][kHD];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const size_t head = blockIdx.x;
    T* kh = kc + head * (size_t)window * kHD;
    T* vh = vc + head * (size_t)window * kHD;
    const int slot = pos % window;
    const int nvalid = min(pos + 1, window);          // before the ring is full, slots 0..pos are the valid ones

    // Every global load of the step is issued before anything is consumed: this thread's key row
    // and its (up to 8) value rows.  The new token's row is taken from the k, v inputs, so the loads
    // do not wait for the cache update below.
    const int cg = tid & 7, jg = tid >> 3;
    Raw8<T> kx[kHD / 8];
    if (tid < nvalid) {
        const T* kr = (tid == slot) ? k + head * kHD : kh + (size_t)tid * kHD;
#pragma unroll
        for (int m = 0; m < kHD / 8; ++m) kx[m].load(kr + m * 8);
    }
    Raw8<T> vx[VROWS];
#pragma unroll
    for (int u = 0; u < VROWS; ++u) {
        const int j = jg + 16 * u;
        if (j < nvalid) {
            const T* vr = (j == slot) ? v + head * kHD : vh + (size_t)j * kHD;
            vx[u].load(vr + cg * 8);
        }
    }
    // cache update, and q to shared memory
    if (tid < kHD) {
        kh[(size_t)slot * kHD + tid] = k[head * kHD + tid];
        s_q[tid] = to_f32(q[head * kHD + tid]) * scale;
    } else {
        vh[(size_t)slot * kHD + tid - kHD] = v[head * kHD + tid - kHD];
    }
    __syncthreads();

    // scores: thread j <-> cached key j
    float s = -INFINITY;
    if (tid < nvalid) {
        float a = 0.f;
#pragma unroll
        for (int m = 0; m < kHD / 8; ++m) {
            float x[8];
            kx[m].get(x);
#pragma unroll
            for (int i = 0; i < 8; ++i) a = fmaf(x[i], s_q[m * 8 + i], a);
        }
        s = a;
    }
    float mx = s;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (lane == 0) s_red[warp] = mx;
    __syncthreads();
    mx = fmaxf(fmaxf(s_red[0], s_red[1]), fmaxf(s_red[2], s_red[3]));
    const float e = tid < nvalid ? expf(s - mx) : 0.f;
    s_p[tid] = e;
    float sum = e;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) s_red[4 + warp] = sum;
    __syncthreads();
    sum = s_red[4] + s_red[5] + s_red[6] + s_red[7];

    // weighted sum of the cached values: 8 threads per row (8 columns each), 16 row groups
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll
    for (int u = 0; u < VROWS; ++u) {
        const int j = jg + 16 * u;
        if (j < nvalid) {
            const float pj = s_p[j];
            float x[8];
            vx[u].get(x);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = fmaf(pj, x[i], acc[i]);
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) s_acc[jg][cg * 8 + i] = acc[i];
    __syncthreads();
    if (tid < kHD) {
        float a = 0.f;
#pragma unroll
        for (int g = 0; g < 16; ++g) a += s_acc[g][tid];
        out[head * kHD + tid] = from_f32<T>(a / sum);
    }
}

template <typename T>
static void launch_t(const void* q, const void* k, const void* v, void* kc, void* vc, void* out, int BH, int window,
                     int pos, float scale, cudaStream_t stream) {
    const T* qq = static_cast<const T*>(q);
    const T* kk = static_cast<const T*>(k);
    const T* vv = static_cast<const T*>(v);
    T* kcc = static_cast<T*>(kc);
    T* vcc = static_cast<T*>(vc);
    T* oo = static_cast<T*>(out);
    if (window <= 64) swa_decode_kernel<T, 4><<<BH, 128, 0, stream>>>(qq, kk, vv, kcc, vcc, oo, window, pos, scale);
    else swa_decode_kernel<T, 8><<<BH, 128, 0, stream>>>(qq, kk, vv, kcc, vcc, oo, window, pos, scale);
}

based_status launch_swa_decode(const void* q, const void* k, const void* v, void* kc, void* vc, void* out, int BH,
                               int window, int pos, float scale, based_dtype io, cudaStream_t stream) {
    if (io == BASED_F32) launch_t<float>(q, k, v, kc, vc, out, BH, window, pos, scale, stream);
    else launch_t<__nv_bfloat16>(q, k, v, kc, vc, out, BH, window, pos, scale, stream);
    note_launch();
    return check_launch("swa_decode_kernel");
}

}  // namespace based
