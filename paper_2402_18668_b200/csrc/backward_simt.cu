// based_prefill_backward: gradients of the causal Taylor linear attention (definition form,
// left-hand side of Eq. (2) of Sec. 4.1) with respect to q, k, v.  The paper gives no backward
// algorithm; this is the chain rule on the definition, evaluated tile by tile in the quadratic
// ("attention") form with fp32 FMAs, a first correct path and not a tensor-core kernel:
//
//   y_i = N_i / D_i,  N_i = sum_{j<=i} w_ij v_j,  D_i = sum_{j<=i} w_ij + eps,  w_ij = 1 + s/4 + s^2/32,
//   s = q_i.k_j;  with G_i the gradient of the loss with respect to y_i:
//   a_i = G_i / D_i,  b_i = -(G_i.y_i) / D_i = -(G_i.N_i) / D_i^2,  ds_ij = (a_i.v_j + b_i)(1/4 + s_ij/16),
//   dq_i = sum_{j<=i} ds_ij k_j,   dk_j = sum_{i>=j} ds_ij q_i,   dv_j = sum_{i>=j} w_ij a_i.
//
// Three launches over 64 x 64 tiles of (query, key) pairs, 128 threads per tile, each thread
// 4 x 8 pairs in registers:
//   row statistics  1/D_i and b_i (from the fp32 numerator)  (grid: query tiles)
//   dq              loops over the key tiles j <= i        (grid: query tiles)
//   dk, dv          loops over the query tiles i >= j      (grid: key tiles); dv as a second phase,
//                   a small matrix product of the tile's weights (through shared memory) with a.
// Arithmetic is O(L^2 (2 d' + 2 d_v)) per head: bound by the fp32 pipe, for sequences up to a few
// thousand tokens about the cost of the linear-time recurrence.
#include "common.cuh"

namespace based {

namespace {
constexpr int kT = 64;             // tile edge (queries and keys)
constexpr int kBT = 128;           // threads per block: 16 row groups (4 rows) x 8 column lanes (8 strided columns)
constexpr int kQP = kDFeat + 1;    // padded row length of q/k tiles (bank-conflict free)

template <int DV> struct BwdSmem {
    float q[kT][kQP];              // query rows of the tile (dq, stats) or of the current query tile (dk/dv)
    float k[kT][kQP];
    float v[kT][DV + 1];
    float a[kT][DV + 1];           // G_i / D_i
    float b[kT];                   // -(G_i.y_i) / D_i
    float w[kT][kT + 1];           // weights of the current tile, [key][query] (dk/dv kernel only)
};

// rows [r0, r0 + 64) of a [L, W] matrix of one head -> fp32 shared tile, zero past the end, optional row scale
template <typename T, int W, int P>
__device__ __forceinline__ void load_tile(const T* __restrict__ src, int r0, int L, float (*dst)[P],
                                          const float* __restrict__ row_scale, int scale_stride) {
    for (int i = threadIdx.x; i < kT * W; i += kBT) {
        const int r = i / W, c = i - r * W;
        float x = 0.f;
        if (r0 + r < L) {
            x = to_f32(src[(size_t)(r0 + r) * W + c]);
            if (row_scale) x *= row_scale[(size_t)(r0 + r) * scale_stride];
        }
        dst[r][c] = x;
    }
}

// s[r][n] = q_row(ty*4+r) . k_row(tx+8n) for this thread's 4 x 8 pairs
__device__ __forceinline__ void pair_scores(const float (*qs)[kQP], const float (*ks)[kQP], int ty, int tx,
                                            float (&s)[4][8]) {
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int n = 0; n < 8; ++n) s[r][n] = 0.f;
#pragma unroll
    for (int m = 0; m < kDFeat; ++m) {
        float qa[4], kb[8];
#pragma unroll
        for (int r = 0; r < 4; ++r) qa[r] = qs[ty * 4 + r][m];
#pragma unroll
        for (int n = 0; n < 8; ++n) kb[n] = ks[tx + 8 * n][m];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int n = 0; n < 8; ++n) s[r][n] = fmaf(qa[r], kb[n], s[r][n]);
    }
}

// g[r][n] = a_row(rows) . v_row(cols) over DV
template <int DV>
__device__ __forceinline__ void pair_av(const float (*as)[DV + 1], const float (*vs)[DV + 1], const int (&ar)[4],
                                        const int (&vr)[8], float (&g)[4][8]) {
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int n = 0; n < 8; ++n) g[r][n] = 0.f;
#pragma unroll 4
    for (int c = 0; c < DV; ++c) {
        float aa[4], vb[8];
#pragma unroll
        for (int r = 0; r < 4; ++r) aa[r] = as[ar[r]][c];
#pragma unroll
        for (int n = 0; n < 8; ++n) vb[n] = vs[vr[n]][c];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int n = 0; n < 8; ++n) g[r][n] = fmaf(aa[r], vb[n], g[r][n]);
    }
}

__device__ __forceinline__ float taylor_w(float s) { return fmaf(s, fmaf(s, 0.03125f, 0.25f), 1.0f); }
__device__ __forceinline__ float taylor_dw(float s) { return fmaf(s, 0.0625f, 0.25f); }
}  // namespace

// stats[i] = (1 / D_i, b_i); numerator-only: (1, 0).  b_i = -(G_i.y_i) / D_i is formed from the fp32
// numerator, -(sum_j w_ij G_i.v_j) / D_i^2, not from the rounded forward output: with few keys in the
// window a_i.v_j + b_i cancels almost completely and a bf16-rounded y would dominate the result.
template <typename T, int DV>
__global__ void __launch_bounds__(kBT) bwd_stats_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                        const T* __restrict__ v, const T* __restrict__ g,
                                                        float2* __restrict__ stats, int L, int numerator_only) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    BwdSmem<DV>& sm = *reinterpret_cast<BwdSmem<DV>*>(smem_raw);
    const int i0 = (gridDim.x - 1 - blockIdx.x) * kT;      // longest loops (last query tiles) first
    const size_t head = blockIdx.y;
    const int ty = threadIdx.x >> 3, tx = threadIdx.x & 7;
    const T* qh = q + head * (size_t)L * kDFeat;
    const T* kh = k + head * (size_t)L * kDFeat;
    float2* st = stats + head * (size_t)L;
    if (numerator_only) {
        for (int i = threadIdx.x; i < kT && i0 + i < L; i += kBT) st[i0 + i] = make_float2(1.f, 0.f);
        return;
    }
    load_tile<T, kDFeat, kQP>(qh, i0, L, sm.q, nullptr, 0);
    load_tile<T, DV, DV + 1>(g + head * (size_t)L * DV, i0, L, sm.a, nullptr, 0);          // G_i, unscaled
    float den[4] = {0.f, 0.f, 0.f, 0.f}, gn[4] = {0.f, 0.f, 0.f, 0.f};
    const int ar[4] = {ty * 4, ty * 4 + 1, ty * 4 + 2, ty * 4 + 3};
    const int vr[8] = {tx, tx + 8, tx + 16, tx + 24, tx + 32, tx + 40, tx + 48, tx + 56};
    for (int j0 = 0; j0 <= i0; j0 += kT) {
        __syncthreads();
        load_tile<T, kDFeat, kQP>(kh, j0, L, sm.k, nullptr, 0);
        load_tile<T, DV, DV + 1>(v + head * (size_t)L * DV, j0, L, sm.v, nullptr, 0);
        __syncthreads();
        float s[4][8], gv[4][8];
        pair_scores(sm.q, sm.k, ty, tx, s);
        pair_av<DV>(sm.a, sm.v, ar, vr, gv);
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int n = 0; n < 8; ++n)
                if (j0 + vr[n] <= i0 + ar[r]) {
                    const float w = taylor_w(s[r][n]);
                    den[r] += w;
                    gn[r] = fmaf(w, gv[r][n], gn[r]);
                }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
#pragma unroll
        for (int o = 1; o < 8; o <<= 1) {
            den[r] += __shfl_xor_sync(0xffffffffu, den[r], o);
            gn[r] += __shfl_xor_sync(0xffffffffu, gn[r], o);
        }
        const int i = i0 + ar[r];
        if (tx == 0 && i < L) {
            const float dinv = 1.0f / (den[r] + kEps);
            st[i] = make_float2(dinv, -gn[r] * dinv * dinv);
        }
    }
}

template <typename T, int DV>
__global__ void __launch_bounds__(kBT) bwd_dq_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                     const T* __restrict__ v, const T* __restrict__ g,
                                                     const float2* __restrict__ stats, T* __restrict__ dq, int L) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    BwdSmem<DV>& sm = *reinterpret_cast<BwdSmem<DV>*>(smem_raw);
    const int i0 = (gridDim.x - 1 - blockIdx.x) * kT;      // longest loops (last query tiles) first
    const size_t head = blockIdx.y;
    const int ty = threadIdx.x >> 3, tx = threadIdx.x & 7;
    const float2* st = stats + head * (size_t)L;
    load_tile<T, kDFeat, kQP>(q + head * (size_t)L * kDFeat, i0, L, sm.q, nullptr, 0);
    load_tile<T, DV, DV + 1>(g + head * (size_t)L * DV, i0, L, sm.a, &st[0].x, 2);       // a_i = G_i / D_i
    for (int i = threadIdx.x; i < kT; i += kBT) sm.b[i] = i0 + i < L ? st[i0 + i].y : 0.f;
    float acc[4][kDFeat];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int m = 0; m < kDFeat; ++m) acc[r][m] = 0.f;
    const int ar[4] = {ty * 4, ty * 4 + 1, ty * 4 + 2, ty * 4 + 3};
    const int vr[8] = {tx, tx + 8, tx + 16, tx + 24, tx + 32, tx + 40, tx + 48, tx + 56};
    for (int j0 = 0; j0 <= i0; j0 += kT) {
        __syncthreads();
        load_tile<T, kDFeat, kQP>(k + head * (size_t)L * kDFeat, j0, L, sm.k, nullptr, 0);
        load_tile<T, DV, DV + 1>(v + head * (size_t)L * DV, j0, L, sm.v, nullptr, 0);
        __syncthreads();
        float s[4][8], gv[4][8];
        pair_scores(sm.q, sm.k, ty, tx, s);
        pair_av<DV>(sm.a, sm.v, ar, vr, gv);
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int n = 0; n < 8; ++n) {
                const bool live = j0 + vr[n] <= i0 + ar[r];
                s[r][n] = live ? (gv[r][n] + sm.b[ar[r]]) * taylor_dw(s[r][n]) : 0.f;          // ds_ij
            }
#pragma unroll
        for (int n = 0; n < 8; ++n)
#pragma unroll
            for (int m = 0; m < kDFeat; ++m) {
                const float kk = sm.k[vr[n]][m];
#pragma unroll
                for (int r = 0; r < 4; ++r) acc[r][m] = fmaf(s[r][n], kk, acc[r][m]);
            }
    }
    T* dqh = dq + head * (size_t)L * kDFeat;
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int m = 0; m < kDFeat; ++m) {
            float x = acc[r][m];
            x += __shfl_xor_sync(0xffffffffu, x, 1);
            x += __shfl_xor_sync(0xffffffffu, x, 2);
            x += __shfl_xor_sync(0xffffffffu, x, 4);
            if (tx == (m & 7) && i0 + ar[r] < L) dqh[(size_t)(i0 + ar[r]) * kDFeat + m] = from_f32<T>(x);
        }
}

template <typename T, int DV>
__global__ void __launch_bounds__(kBT) bwd_dkdv_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                       const T* __restrict__ v, const T* __restrict__ g,
                                                       const float2* __restrict__ stats, T* __restrict__ dk,
                                                       T* __restrict__ dv, int L) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    BwdSmem<DV>& sm = *reinterpret_cast<BwdSmem<DV>*>(smem_raw);
    const int j0 = blockIdx.x * kT;
    const size_t head = blockIdx.y;
    const int ty = threadIdx.x >> 3, tx = threadIdx.x & 7;
    const float2* st = stats + head * (size_t)L;
    // here rows are keys (ty) and columns are queries (tx): pair_scores(k, q) gives s[key][query]
    load_tile<T, kDFeat, kQP>(k + head * (size_t)L * kDFeat, j0, L, sm.k, nullptr, 0);
    load_tile<T, DV, DV + 1>(v + head * (size_t)L * DV, j0, L, sm.v, nullptr, 0);
    float dka[4][kDFeat];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int m = 0; m < kDFeat; ++m) dka[r][m] = 0.f;
    // dv phase: thread (ty, tx) owns keys ty*4..+3 and the DV/8 columns tx, tx+8, ...
    constexpr int NC = DV / 8;
    float dva[4][NC];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < NC; ++c) dva[r][c] = 0.f;
    const int kr[4] = {ty * 4, ty * 4 + 1, ty * 4 + 2, ty * 4 + 3};
    const int qc[8] = {tx, tx + 8, tx + 16, tx + 24, tx + 32, tx + 40, tx + 48, tx + 56};
    for (int i0 = j0; i0 < L; i0 += kT) {
        __syncthreads();
        load_tile<T, kDFeat, kQP>(q + head * (size_t)L * kDFeat, i0, L, sm.q, nullptr, 0);
        load_tile<T, DV, DV + 1>(g + head * (size_t)L * DV, i0, L, sm.a, &st[0].x, 2);
        for (int i = threadIdx.x; i < kT; i += kBT) sm.b[i] = i0 + i < L ? st[i0 + i].y : 0.f;
        __syncthreads();
        float s[4][8], gv[4][8];
        pair_scores(sm.k, sm.q, ty, tx, s);                 // s[key r][query n]
        pair_av<DV>(sm.v, sm.a, kr, qc, gv);                // v_j . a_i
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int n = 0; n < 8; ++n) {
                const bool live = j0 + kr[r] <= i0 + qc[n] && i0 + qc[n] < L;
                const float sv = s[r][n];
                sm.w[kr[r]][qc[n]] = live ? taylor_w(sv) : 0.f;
                s[r][n] = live ? (gv[r][n] + sm.b[qc[n]]) * taylor_dw(sv) : 0.f;               // ds_ij
            }
#pragma unroll
        for (int n = 0; n < 8; ++n)
#pragma unroll
            for (int m = 0; m < kDFeat; ++m) {
                const float qq = sm.q[qc[n]][m];
#pragma unroll
                for (int r = 0; r < 4; ++r) dka[r][m] = fmaf(s[r][n], qq, dka[r][m]);
            }
        __syncthreads();
        // dv_j += sum_i w_ij a_i
#pragma unroll 4
        for (int i = 0; i < kT; ++i) {
            float ww[4], aa[NC];
#pragma unroll
            for (int r = 0; r < 4; ++r) ww[r] = sm.w[kr[r]][i];
#pragma unroll
            for (int c = 0; c < NC; ++c) aa[c] = sm.a[i][tx + 8 * c];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < NC; ++c) dva[r][c] = fmaf(ww[r], aa[c], dva[r][c]);
        }
    }
    T* dkh = dk + head * (size_t)L * kDFeat;
    T* dvh = dv + head * (size_t)L * DV;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int j = j0 + kr[r];
#pragma unroll
        for (int m = 0; m < kDFeat; ++m) {
            float x = dka[r][m];
            x += __shfl_xor_sync(0xffffffffu, x, 1);
            x += __shfl_xor_sync(0xffffffffu, x, 2);
            x += __shfl_xor_sync(0xffffffffu, x, 4);
            if (tx == (m & 7) && j < L) dkh[(size_t)j * kDFeat + m] = from_f32<T>(x);
        }
        if (j < L)
#pragma unroll
            for (int c = 0; c < NC; ++c) dvh[(size_t)j * DV + tx + 8 * c] = from_f32<T>(dva[r][c]);
    }
}

template <typename T, int DV>
static based_status launch_t(const void* q, const void* k, const void* v, const void* g, void* dq, void* dk,
                             void* dv, float* stats, int BH, int L, int numerator_only, cudaStream_t stream) {
    const size_t smem = sizeof(BwdSmem<DV>);
    {
        static bool configured[64] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BASED_ERR_CUDA;
        std::lock_guard<std::mutex> lock(setup_mutex());
        if (!configured[dev]) {
            if (cudaFuncSetAttribute(bwd_stats_kernel<T, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                    cudaSuccess ||
                cudaFuncSetAttribute(bwd_dq_kernel<T, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                    cudaSuccess ||
                cudaFuncSetAttribute(bwd_dkdv_kernel<T, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                    cudaSuccess)
                return BASED_ERR_CUDA;
            configured[dev] = true;
        }
    }
    const dim3 grid((L + kT - 1) / kT, BH);
    const T* qq = static_cast<const T*>(q);
    const T* kk = static_cast<const T*>(k);
    const T* vv = static_cast<const T*>(v);
    const T* gg = static_cast<const T*>(g);
    float2* st = reinterpret_cast<float2*>(stats);
    bwd_stats_kernel<T, DV><<<grid, kBT, smem, stream>>>(qq, kk, vv, gg, st, L, numerator_only);
    note_launch();
    based_status s = check_launch("bwd_stats_kernel");
    if (s != BASED_OK) return s;
    bwd_dq_kernel<T, DV><<<grid, kBT, smem, stream>>>(qq, kk, vv, gg, st, static_cast<T*>(dq), L);
    note_launch();
    s = check_launch("bwd_dq_kernel");
    if (s != BASED_OK) return s;
    bwd_dkdv_kernel<T, DV><<<grid, kBT, smem, stream>>>(qq, kk, vv, gg, st, static_cast<T*>(dk), static_cast<T*>(dv), L);
    note_launch();
    return check_launch("bwd_dkdv_kernel");
}

based_status launch_prefill_backward(const void* q, const void* k, const void* v, const void* g, void* dq, void* dk,
                                     void* dv, float* stats, int BH, int L, int d_v, based_dtype io,
                                     int numerator_only, cudaStream_t stream) {
    if (io == BASED_F32) {
        if (d_v == 64) return launch_t<float, 64>(q, k, v, g, dq, dk, dv, stats, BH, L, numerator_only, stream);
        if (d_v == 112) return launch_t<float, 112>(q, k, v, g, dq, dk, dv, stats, BH, L, numerator_only, stream);
        return launch_t<float, 128>(q, k, v, g, dq, dk, dv, stats, BH, L, numerator_only, stream);
    }
    if (d_v == 64) return launch_t<__nv_bfloat16, 64>(q, k, v, g, dq, dk, dv, stats, BH, L, numerator_only, stream);
    if (d_v == 112) return launch_t<__nv_bfloat16, 112>(q, k, v, g, dq, dk, dv, stats, BH, L, numerator_only, stream);
    return launch_t<__nv_bfloat16, 128>(q, k, v, g, dq, dk, dv, stats, BH, L, numerator_only, stream);
}

}  // namespace based
