// Device-side body of the linear-attention decode step (shared by decode.cu and generation_step.cu).
#pragma once
#include "common.cuh"

namespace based {

// STREAM: the state of all heads together is larger than L2, so every line is used exactly once
// per step: load and store it with the evict-first (streaming) policy.  Measured on B200 at batch
// 128 x 16 heads, d_v 128: 94.4 us per step against 96.9 us with the default policy.
// SYM: the state holds the 153 symmetric features (one per unordered pair, the feature count of the
// appendix "Computing Recurrent State Size") instead of the 273 of the full outer product: the
// same outputs from 44 % fewer state bytes per step.
// The body is a device function of a 256-thread CTA for head `head`, so that the fused generation step
// (both mixers in one launch) runs the same code as the stand-alone kernel.
template <int DV, typename T, bool STREAM, bool SYM>
__device__ __forceinline__ void decode_step_body(const T* __restrict__ q, const T* __restrict__ k,
                                                 const T* __restrict__ v, float* __restrict__ kv,
                                                 float* __restrict__ z, T* __restrict__ out, int numerator_only,
                                                 size_t head) {
    constexpr int TPR = DV / 4;                    // threads per state row (one float4 each)
    constexpr int RPP = 256 / TPR;                 // rows per pass: 8 (d_v 128) or 16 (d_v 64)
    constexpr int ND = SYM ? kDSym : kD;           // state rows
    constexpr int UNROLL = SYM ? 5 : (DV == 64) ? 6 : 7;    // loads in flight per thread (35 = 5*7, 18 = 3*6, 20 = 4*5)
    // full: 35 or 18 passes; symmetric: 20 or 10; d_v 112 (28 threads per row, 9 rows per pass, the last
    // 4 threads idle): 31 and 17 passes, rounded up to the unroll factor (rows past the end are skipped)
    constexpr int NPASS = ((ND + RPP - 1) / RPP + UNROLL - 1) / UNROLL * UNROLL;
    constexpr int DPAD = NPASS * RPP;

    __shared__ float s_x[2][kDFeat];
    __shared__ float s_pq[DPAD], s_pk[DPAD];
    __shared__ __align__(16) float s_num[RPP][DV];
    __shared__ float s_den[8];

    const int tid = threadIdx.x;
    const int c4 = tid % TPR, rslot = tid / TPR;
    const bool row_thread = rslot < RPP;             // false only for the idle tail threads of d_v 112

    if (tid < kDFeat) s_x[0][tid] = to_f32(q[head * kDFeat + tid]);
    else if (tid < 2 * kDFeat) s_x[1][tid - kDFeat] = to_f32(k[head * kDFeat + tid - kDFeat]);
    float vv[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) vv[e] = to_f32(v[head * DV + c4 * 4 + e]);
    __syncthreads();
    for (int f = tid; f < DPAD; f += 256) {
        s_pq[f] = f < ND ? (SYM ? psi_at(s_x[0], f) : phi_at(s_x[0], f)) : 0.f;
        s_pk[f] = f < ND ? (SYM ? psi_at(s_x[1], f) : phi_at(s_x[1], f)) : 0.f;
    }
    __syncthreads();

    // K-state update and denominator phi(q).z
    float dpart = 0.f;
    float* zh = z + head * ND;
    for (int f = tid; f < ND; f += 256) {
        const float zn = zh[f] + s_pk[f];
        zh[f] = zn;
        dpart = fmaf(s_pq[f], zn, dpart);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dpart += __shfl_xor_sync(0xffffffffu, dpart, o);
    if ((tid & 31) == 0) s_den[tid >> 5] = dpart;

    // KV-state stream: S[r, :] += phi(k)[r] * v ; num += phi(q)[r] * S[r, :]
    float4* S = reinterpret_cast<float4*>(kv + head * (size_t)ND * DV) + c4;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int p0 = 0; p0 < NPASS; p0 += UNROLL) {
        float4 s[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int r = (p0 + u) * RPP + rslot;
            if (r < ND && row_thread) s[u] = STREAM ? __ldcs(&S[(size_t)r * TPR]) : S[(size_t)r * TPR];
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int r = (p0 + u) * RPP + rslot;
            if (r < ND && row_thread) {
                const float pk = s_pk[r], pq = s_pq[r];
                s[u].x = fmaf(pk, vv[0], s[u].x);
                s[u].y = fmaf(pk, vv[1], s[u].y);
                s[u].z = fmaf(pk, vv[2], s[u].z);
                s[u].w = fmaf(pk, vv[3], s[u].w);
                acc.x = fmaf(pq, s[u].x, acc.x);
                acc.y = fmaf(pq, s[u].y, acc.y);
                acc.z = fmaf(pq, s[u].z, acc.z);
                acc.w = fmaf(pq, s[u].w, acc.w);
                if (STREAM) __stcs(&S[(size_t)r * TPR], s[u]);
                else S[(size_t)r * TPR] = s[u];
            }
        }
    }
    if (row_thread) *reinterpret_cast<float4*>(&s_num[rslot][c4 * 4]) = acc;
    __syncthreads();
    if (tid < DV) {
        float num = 0.f;
#pragma unroll
        for (int r = 0; r < RPP; ++r) num += s_num[r][tid];
        float den = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) den += s_den[w];
        out[head * DV + tid] = from_f32<T>(numerator_only ? num : num / (den + kEps));
    }
}


}  // namespace based
