// Device-side body of the sliding-window decode step (shared by swa_decode.cu and generation_step.cu).
#pragma once
#include <math.h>

#include "common.cuh"
#include "sm100.cuh"

namespace based {
namespace swa_dec {
constexpr int kHD = 64;
constexpr int kWarps = 4;

// Per-warp partial results (flash-style: each warp works relative to the maximum of its own rows
// and the partials are rescaled when they are combined).
struct Partials {
    float acc[kWarps][kHD];
    float mx[kWarps];
    float sum[kWarps];
};

// The 8 columns lane-slot c owns in a 64-wide row: one 16-byte piece of a bf16 row, two 16-byte
// pieces (32 columns apart) of an fp32 row, so that a warp always reads consecutive 16-byte words.
template <typename T> struct Cols;
template <> struct Cols<__nv_bfloat16> {
    static __device__ __forceinline__ int col(int c, int i) { return c * 8 + i; }
    static __device__ __forceinline__ void load(const __nv_bfloat16* row, int c, float (&x)[8]) {
        const uint4 u = *reinterpret_cast<const uint4*>(row + c * 8);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __bfloat1622float2(h[i]);
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* row, int c, const float (&x)[8]) {
        uint4 u;
        __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&u);
#pragma unroll
        for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
        *reinterpret_cast<uint4*>(row + c * 8) = u;
    }
};
template <> struct Cols<float> {
    static __device__ __forceinline__ int col(int c, int i) { return i < 4 ? c * 4 + i : 32 + c * 4 + i - 4; }
    static __device__ __forceinline__ void load(const float* row, int c, float (&x)[8]) {
        const float4 a = *reinterpret_cast<const float4*>(row + c * 4);
        const float4 b = *reinterpret_cast<const float4*>(row + 32 + c * 4);
        x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
    }
    static __device__ __forceinline__ void store(float* row, int c, const float (&x)[8]) {
        *reinterpret_cast<float4*>(row + c * 4) = make_float4(x[0], x[1], x[2], x[3]);
        *reinterpret_cast<float4*>(row + 32 + c * 4) = make_float4(x[4], x[5], x[6], x[7]);
    }
};

// Shared memory: K rows [window][64], V rows [window][64], new q, k, v [64] each (all of type T),
// then the mbarrier, the give-up flag of the bounded wait, and the warps' partial results.
template <typename T>
size_t swa_decode_smem_bytes(int window) {
    return ((size_t)2 * window * kHD + 3 * kHD) * sizeof(T) + 16 + sizeof(Partials);
}


// One head's step by a group of 128 threads (tid = index within the group, BAR = the group's named
// barrier, smem = the group's shared memory).  n_tickets: in advance mode, how many groups take a ticket.
template <typename T, int NPW, int BAR>     // NPW >= ceil(window / (4 * kWarps)): passes of 4 rows per warp
__device__ __forceinline__ void swa_decode_body(const T* __restrict__ q, const T* __restrict__ k,
                                                const T* __restrict__ v, T* __restrict__ kc, T* __restrict__ vc,
                                                T* __restrict__ out, int window, int pos_arg, const int* pos_dev,
                                                int* pos_adv, float scale, unsigned int* __restrict__ error_word,
                                                size_t head, int tid, int n_tickets, unsigned char* smem, int pos_group = 0) {
    auto group_sync = [&]() { asm volatile("bar.sync %0, 128;" ::"n"(BAR) : "memory"); };
    // the position comes from device memory when the launch is part of a captured graph that is
    // replayed as the sequence grows.  In advance mode pos_dev and pos_adv name the same word, which
    // the last CTA rewrites at its end: no restrict on either, and the read is a volatile one
    // pos_group > 0: one position per sequence (pos_dev[b], b = head / pos_group) for batches whose sequences
    // have different lengths
    const int pos = pos_dev ? *reinterpret_cast<const volatile int*>(pos_dev + (pos_group > 0 ? head / pos_group : 0)) : pos_arg;
    T* s_K = reinterpret_cast<T*>(smem);
    T* s_V = s_K + (size_t)window * kHD;
    T* s_qn = s_V + (size_t)window * kHD;
    T* s_kn = s_qn + kHD;
    T* s_vn = s_kn + kHD;
    uint64_t* bar = reinterpret_cast<uint64_t*>(s_vn + kHD);
    volatile uint32_t* give_up = reinterpret_cast<volatile uint32_t*>(bar + 1);
    Partials& part = *reinterpret_cast<Partials*>(bar + 2);

    const int lane = tid & 31, warp = tid >> 5, g = lane >> 3, c = lane & 7;
    T* kh = kc + head * (size_t)window * kHD;
    T* vh = vc + head * (size_t)window * kHD;
    const int slot = pos % window;
    const int nvalid = min(pos + 1, window);          // before the ring is full, slots 0..pos are the valid ones

    if (tid == 0) {
        sm100::mbar_init(bar, 1);
        *give_up = 0;
        sm100::fence_mbar_init();
        const uint32_t rows = (uint32_t)nvalid * kHD * sizeof(T), one = kHD * sizeof(T);
        sm100::mbar_arrive_expect_tx(bar, 2 * rows + 3 * one);
        sm100::bulk_load_1d(s_K, kh, rows, bar);
        sm100::bulk_load_1d(s_V, vh, rows, bar);
        sm100::bulk_load_1d(s_qn, q + head * kHD, one, bar);
        sm100::bulk_load_1d(s_kn, k + head * kHD, one, bar);
        sm100::bulk_load_1d(s_vn, v + head * kHD, one, bar);
    }
    group_sync();
    if (!sm100::mbar_wait(bar, 0, give_up)) {
        // gave up on the loads: report it, but still take this CTA's ticket, or the position of a replayed
        // graph would stay stuck (and its ticket count off) for every later step
        if (tid == 0) {
            atomicExch(error_word, 1u);
            if (pos_adv != nullptr && atomicAdd(pos_adv + 1, 1) == n_tickets - 1) {
                pos_adv[1] = 0;
                pos_adv[0] = pos + 1;
            }
        }
        return;
    }

    // cache update (warp 0): 16-byte pieces of the new key row, then of the new value row
    if (warp == 0) {
        constexpr int kPieces = kHD * sizeof(T) / 16;          // 8 (bf16) or 16 (fp32) per row
        if (lane < kPieces)
            reinterpret_cast<uint4*>(kh + (size_t)slot * kHD)[lane] = reinterpret_cast<const uint4*>(s_kn)[lane];
        else if (lane < 2 * kPieces)
            reinterpret_cast<uint4*>(vh + (size_t)slot * kHD)[lane - kPieces] =
                reinterpret_cast<const uint4*>(s_vn)[lane - kPieces];
    }

    float qx[8];
    Cols<T>::load(s_qn, c, qx);
#pragma unroll
    for (int i = 0; i < 8; ++i) qx[i] *= scale;

    // scores: pass p of this warp, row group g <-> cached key 4 * (p * kWarps + warp) + g
    float s[NPW];
    float mx = -INFINITY;
#pragma unroll
    for (int p = 0; p < NPW; ++p) {
        const int row = 4 * (p * kWarps + warp) + g;
        float a = 0.f;
        if (row < nvalid) {
            float x[8];
            Cols<T>::load(row == slot ? s_kn : s_K + (size_t)row * kHD, c, x);
#pragma unroll
            for (int i = 0; i < 8; ++i) a = fmaf(x[i], qx[i], a);
        }
        a += __shfl_xor_sync(0xffffffffu, a, 1);
        a += __shfl_xor_sync(0xffffffffu, a, 2);
        a += __shfl_xor_sync(0xffffffffu, a, 4);
        s[p] = row < nvalid ? a : -INFINITY;
        mx = fmaxf(mx, s[p]);
    }
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
    const float ref = mx == -INFINITY ? 0.f : mx;     // a warp whose rows all lie outside the window
    float sum = 0.f;
#pragma unroll
    for (int p = 0; p < NPW; ++p) {
        s[p] = expf(s[p] - ref);                      // exp(-inf) = 0 for rows outside the window
        sum += s[p];
    }
    sum += __shfl_xor_sync(0xffffffffu, sum, 8);
    sum += __shfl_xor_sync(0xffffffffu, sum, 16);

    // this warp's weighted sum of cached values
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll
    for (int p = 0; p < NPW; ++p) {
        const int row = 4 * (p * kWarps + warp) + g;
        if (row < nvalid) {
            float x[8];
            Cols<T>::load(row == slot ? s_vn : s_V + (size_t)row * kHD, c, x);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = fmaf(s[p], x[i], acc[i]);
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 8);
        acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 16);
    }
    if (g == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) part.acc[warp][Cols<T>::col(c, i)] = acc[i];
    }
    if (lane == 0) {
        part.mx[warp] = mx;
        part.sum[warp] = sum;
    }
    group_sync();

    // combine the warps' partials (warp 0 always holds row 0, so the overall maximum is finite)
    if (tid < kHD) {
        float M = part.mx[0];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) M = fmaxf(M, part.mx[w]);
        float num = 0.f, den = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float f = expf(part.mx[w] - M);
            num = fmaf(f, part.acc[w][tid], num);
            den = fmaf(f, part.sum[w], den);
        }
        out[head * kHD + tid] = from_f32<T>(num / den);
    }
    // advance mode: pos_adv = {position, ticket}.  Every CTA read the position at its start and takes a
    // ticket at its end, so the CTA that takes the last one knows that all of them have read it: it
    // resets the ticket and stores position + 1 for the next launch
    if (pos_adv != nullptr && tid == 0) {
        if (atomicAdd(pos_adv + 1, 1) == n_tickets - 1) {
            pos_adv[1] = 0;
            pos_adv[0] = pos + 1;
        }
    }
}

}  // namespace swa_dec
}  // namespace based
