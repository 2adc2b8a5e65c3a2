// baseconv_gate_forward / baseconv_gate_step: the gated short convolution at the core of the
// BaseConv layer (App. "Extended Architecture Details", paragraph "Convolution"):
//
//   out[b,i,c] = a[b,i,c] * SiLU( sum_{j<w, j<=i} h[j,c] * g[b,i-j,c] + b2[c] )
//
// a = u W1 + b1 and g = u W2 are the layer's two up-projections (plain matrix products, not
// part of this file); h is the depthwise causal filter of width w (the paper suggests 3), h[0]
// the tap on the current token.
//
// The op is one pass over a, g and out: 3 elements of traffic per output element and a dozen
// flops, so it is bound by HBM bandwidth.  A thread owns 8 consecutive channels (one 16-byte
// piece of a bf16 row, two of an fp32 row) and walks a run of kRun tokens with the last w-1 rows
// of g in registers, so g is read once (plus w-1 halo rows per run, which the neighbouring run
// has just brought into L2); a warp covers 256 consecutive channels of a row.  The loop is
// software-pipelined: the rows of the next four tokens are in flight (kept packed, as loaded)
// while the current four are converted, combined and stored.
#include "common.cuh"

namespace based {

namespace {
constexpr int kRun = 64;        // tokens per thread run
constexpr int kUnroll = 4;      // tokens whose loads are in flight together
constexpr int kThreadsBC = 128;

template <typename T> struct Row8;
template <> struct Row8<__nv_bfloat16> {
    struct Raw { uint4 u; };
    static __device__ __forceinline__ void load_raw(const __nv_bfloat16* p, Raw& r) {
        r.u = __ldcs(reinterpret_cast<const uint4*>(p));
    }
    static __device__ __forceinline__ void unpack(const Raw& r, float (&x)[8]) {
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&r.u);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __bfloat1622float2(h[i]);
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
        }
    }
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&x)[8]) {
        const uint4 u = __ldcs(reinterpret_cast<const uint4*>(p));
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __bfloat1622float2(h[i]);
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&x)[8]) {
        uint4 u;
        __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&u);
#pragma unroll
        for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
        __stcs(reinterpret_cast<uint4*>(p), u);
    }
};
template <> struct Row8<float> {
    struct Raw { float4 a, b; };
    static __device__ __forceinline__ void load_raw(const float* p, Raw& r) {
        r.a = __ldcs(reinterpret_cast<const float4*>(p));
        r.b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
    }
    static __device__ __forceinline__ void unpack(const Raw& r, float (&x)[8]) {
        x[0] = r.a.x; x[1] = r.a.y; x[2] = r.a.z; x[3] = r.a.w; x[4] = r.b.x; x[5] = r.b.y; x[6] = r.b.z; x[7] = r.b.w;
    }
    static __device__ __forceinline__ void load(const float* p, float (&x)[8]) {
        const float4 a = __ldcs(reinterpret_cast<const float4*>(p)), b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
        x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
    }
    static __device__ __forceinline__ void store(float* p, const float (&x)[8]) {
        __stcs(reinterpret_cast<float4*>(p), make_float4(x[0], x[1], x[2], x[3]));
        __stcs(reinterpret_cast<float4*>(p) + 1, make_float4(x[4], x[5], x[6], x[7]));
    }
};

// SiLU(x) = x * sigmoid(x); the fast exponential and division are exact enough for bf16 outputs,
// fp32 io takes the accurate ones
template <bool FAST>
__device__ __forceinline__ float silu(float x) {
    return FAST ? __fdividef(x, 1.0f + __expf(-x)) : x / (1.0f + expf(-x));
}
}  // namespace

template <typename T, int W>
__global__ void __launch_bounds__(kThreadsBC) baseconv_gate_kernel(const T* __restrict__ a, const T* __restrict__ g,
                                                                   const float* __restrict__ h,
                                                                   const float* __restrict__ b2, T* __restrict__ out,
                                                                   int N, int C) {
    constexpr bool FAST = sizeof(T) == 2;
    const int c0 = (blockIdx.x * kThreadsBC + threadIdx.x) * 8;
    if (c0 >= C) return;
    const int i0 = blockIdx.y * kRun;
    const int i1 = min(N, i0 + kRun);
    const size_t base = (size_t)blockIdx.z * N * C + c0;

    float taps[W][8], bias[8];
#pragma unroll
    for (int j = 0; j < W; ++j)
#pragma unroll
        for (int e = 0; e < 8; ++e) taps[j][e] = h[(size_t)j * C + c0 + e];
#pragma unroll
    for (int e = 0; e < 8; ++e) bias[e] = b2[c0 + e];

    // prev[j] = g of the token j+1 steps back (zero before the sequence start)
    float prev[W > 1 ? W - 1 : 1][8];
#pragma unroll
    for (int j = 0; j < W - 1; ++j) {
        const int i = i0 - 1 - j;
        if (i >= 0) Row8<T>::load(g + base + (size_t)i * C, prev[j]);
        else {
#pragma unroll
            for (int e = 0; e < 8; ++e) prev[j][e] = 0.f;
        }
    }

    // software pipeline: the loads of the next kUnroll tokens are in flight while these are used
    typename Row8<T>::Raw gr[kUnroll], ar[kUnroll], gn[kUnroll], an[kUnroll];
    auto fetch = [&](int i, typename Row8<T>::Raw (&gq)[kUnroll], typename Row8<T>::Raw (&aq)[kUnroll]) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (i + u < i1) {
                Row8<T>::load_raw(g + base + (size_t)(i + u) * C, gq[u]);
                Row8<T>::load_raw(a + base + (size_t)(i + u) * C, aq[u]);
            }
        }
    };
    fetch(i0, gr, ar);
    for (int i = i0; i < i1; i += kUnroll) {
        fetch(i + kUnroll, gn, an);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (i + u < i1) {
                float gx[8], ax[8], y[8];
                Row8<T>::unpack(gr[u], gx);
                Row8<T>::unpack(ar[u], ax);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    float acc = fmaf(taps[0][e], gx[e], bias[e]);
#pragma unroll
                    for (int j = 1; j < W; ++j) acc = fmaf(taps[j][e], prev[j - 1][e], acc);
                    y[e] = ax[e] * silu<FAST>(acc);
                }
                Row8<T>::store(out + base + (size_t)(i + u) * C, y);
#pragma unroll
                for (int j = W - 2; j >= 1; --j)
#pragma unroll
                    for (int e = 0; e < 8; ++e) prev[j][e] = prev[j - 1][e];
                if (W > 1) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) prev[0][e] = gx[e];
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            gr[u] = gn[u];
            ar[u] = an[u];
        }
    }
}

// One token: state [B, W-1, C], row j = g of the token j+1 steps back; shifted in place.
template <typename T, int W>
__global__ void __launch_bounds__(kThreadsBC) baseconv_step_kernel(const T* __restrict__ a, const T* __restrict__ g,
                                                                   const float* __restrict__ h,
                                                                   const float* __restrict__ b2, T* __restrict__ state,
                                                                   T* __restrict__ out, int C) {
    constexpr bool FAST = sizeof(T) == 2;
    const int c0 = (blockIdx.x * kThreadsBC + threadIdx.x) * 8;
    if (c0 >= C) return;
    const size_t b = blockIdx.y;
    T* st = state + b * (size_t)(W - 1) * C + c0;
    float gx[8], ax[8], acc[8], prev[W > 1 ? W - 1 : 1][8];
    Row8<T>::load(g + b * C + c0, gx);
    Row8<T>::load(a + b * C + c0, ax);
#pragma unroll
    for (int j = 0; j < W - 1; ++j) Row8<T>::load(st + (size_t)j * C, prev[j]);
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = fmaf(h[c0 + e], gx[e], b2[c0 + e]);
#pragma unroll
    for (int j = 1; j < W; ++j)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = fmaf(h[(size_t)j * C + c0 + e], prev[j - 1][e], acc[e]);
    float y[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) y[e] = ax[e] * silu<FAST>(acc[e]);
    Row8<T>::store(out + b * C + c0, y);
#pragma unroll
    for (int j = W - 2; j >= 1; --j) Row8<T>::store(st + (size_t)j * C, prev[j - 1]);
    if (W > 1) Row8<T>::store(st, gx);
}

template <typename T, int W>
static void launch_w(const void* a, const void* g, const float* h, const float* b2, void* state, void* out, int B,
                     int N, int C, bool step, cudaStream_t stream) {
    const int gx = (C / 8 + kThreadsBC - 1) / kThreadsBC;
    if (step)
        baseconv_step_kernel<T, W><<<dim3(gx, B), kThreadsBC, 0, stream>>>(
            static_cast<const T*>(a), static_cast<const T*>(g), h, b2, static_cast<T*>(state), static_cast<T*>(out), C);
    else
        baseconv_gate_kernel<T, W><<<dim3(gx, (N + kRun - 1) / kRun, B), kThreadsBC, 0, stream>>>(
            static_cast<const T*>(a), static_cast<const T*>(g), h, b2, static_cast<T*>(out), N, C);
}

template <typename T>
static void launch_t(const void* a, const void* g, const float* h, const float* b2, void* state, void* out, int B,
                     int N, int C, int width, bool step, cudaStream_t stream) {
    switch (width) {
        case 1: launch_w<T, 1>(a, g, h, b2, state, out, B, N, C, step, stream); break;
        case 2: launch_w<T, 2>(a, g, h, b2, state, out, B, N, C, step, stream); break;
        case 3: launch_w<T, 3>(a, g, h, b2, state, out, B, N, C, step, stream); break;
        default: launch_w<T, 4>(a, g, h, b2, state, out, B, N, C, step, stream); break;
    }
}

based_status launch_baseconv(const void* a, const void* g, const float* h, const float* b2, void* state, void* out,
                             int B, int N, int C, int width, bool step, based_dtype io, cudaStream_t stream) {
    if (io == BASED_F32) launch_t<float>(a, g, h, b2, state, out, B, N, C, width, step, stream);
    else launch_t<__nv_bfloat16>(a, g, h, b2, state, out, B, N, C, width, step, stream);
    note_launch();
    return check_launch(step ? "baseconv_step_kernel" : "baseconv_gate_kernel");
}

}  // namespace based
