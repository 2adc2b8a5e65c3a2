// Feature dimensions other than 16: d' in {8, 24, 32} (the paper's feature-map ablation trains
// Taylor maps of dimension 8, 16, 24 and 32, i.e. 73, 273, 601 and 1057 expanded features).
// The fp32 FMA paths (fp32 io; with bf16 io the outputs from the empty state and the final state run
// on tensor cores instead: the tile kernel's forward mode and generic_state_tc.cu):
//
//   prefill   the definition form of Eq. (2), Sec. 4.1, tile by tile: 64 queries per CTA loop over
//             the key tiles j <= i; scores (any d'), weights w = 1 + s/sqrt(d') + s^2/(2 d'), row
//             sums, and the product of the weight tile (through shared memory) with the value
//             tile.  A given initial state adds phi(q_i).S0 and phi(q_i).z0 per row.
//   state     S = S0 + sum_j phi(k_j) v_j^T, z = z0 + sum_j phi(k_j): one CTA per (head, 32 features).
//   decode    the recurrent step as a stream over the [D, d_v] state, D = 1 + d' + d'^2 (both io dtypes; the
//             loop of the d' = 16 decode kernel with the number of rows as a parameter).
//
// The state layout is the 273-row layout's generalisation: constant, linear terms, row-major
// outer product.  The chunked tensor-core prefill and the symmetric format exist for d' = 16 only.
#include "common.cuh"

namespace based {

namespace {
constexpr int kT = 64;             // tile edge
constexpr int kBT = 128;           // threads: 16 row groups (4 rows) x 8 column lanes
constexpr int kMaxDF = 32;
constexpr int kQP = kMaxDF + 1;    // padded row length of q/k tiles

__host__ __device__ constexpr int expanded_dim(int df) { return 1 + df + df * df; }

struct FeatScale { float lin, quad, s1, s2; };      // x/d'^(1/4), x x/(sqrt2 sqrt d'), s/sqrt d', s^2/(2 d')
__device__ __forceinline__ FeatScale feat_scale(int df) {
    const float rd = sqrtf((float)df);
    return {rsqrtf(rd), 1.0f / (1.41421356237309505f * rd), 1.0f / rd, 0.5f / (float)df};
}
// expanded feature f of x[df]
__device__ __forceinline__ float phi_gen(const float* x, int df, int f, const FeatScale& sc) {
    if (f == 0) return 1.0f;
    if (f <= df) return x[f - 1] * sc.lin;
    const int p = f - 1 - df;
    return x[p / df] * x[p % df] * sc.quad;
}

template <int DV> struct FwdSmem {
    float q[kT][kQP];
    float k[kT][kQP];
    float v[kT][DV + 1];
    float w[kT][kT + 1];           // weights of the current tile [query][key]
};

template <typename T>
__device__ __forceinline__ void load_rows(const T* __restrict__ src, int r0, int L, int W, float* dst, int pitch) {
    for (int i = threadIdx.x; i < kT * W; i += kBT) {
        const int r = i / W, c = i - r * W;
        dst[r * pitch + c] = r0 + r < L ? to_f32(src[(size_t)(r0 + r) * W + c]) : 0.f;
    }
}
}  // namespace

template <typename T, int DV>
__global__ void __launch_bounds__(kBT) generic_prefill_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                              const T* __restrict__ v, T* __restrict__ out,
                                                              const float* __restrict__ kv0,
                                                              const float* __restrict__ z0, int L, int df,
                                                              int numerator_only) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    FwdSmem<DV>& sm = *reinterpret_cast<FwdSmem<DV>*>(smem_raw);
    const int i0 = (gridDim.x - 1 - blockIdx.x) * kT;       // longest loops first
    const size_t head = blockIdx.y;
    const int ty = threadIdx.x >> 3, tx = threadIdx.x & 7;
    const FeatScale sc = feat_scale(df);
    const int D = expanded_dim(df);
    constexpr int NC = DV / 8;
    load_rows<T>(q + head * (size_t)L * df, i0, L, df, &sm.q[0][0], kQP);
    float num[4][NC], den[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < NC; ++c) num[r][c] = 0.f;
    for (int j0 = 0; j0 <= i0; j0 += kT) {
        __syncthreads();
        load_rows<T>(k + head * (size_t)L * df, j0, L, df, &sm.k[0][0], kQP);
        load_rows<T>(v + head * (size_t)L * DV, j0, L, DV, &sm.v[0][0], DV + 1);
        __syncthreads();
        float s[4][8];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int n = 0; n < 8; ++n) s[r][n] = 0.f;
        for (int m = 0; m < df; ++m) {
            float qa[4], kb[8];
#pragma unroll
            for (int r = 0; r < 4; ++r) qa[r] = sm.q[ty * 4 + r][m];
#pragma unroll
            for (int n = 0; n < 8; ++n) kb[n] = sm.k[tx + 8 * n][m];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int n = 0; n < 8; ++n) s[r][n] = fmaf(qa[r], kb[n], s[r][n]);
        }
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int n = 0; n < 8; ++n) {
                const bool live = j0 + tx + 8 * n <= i0 + ty * 4 + r;
                const float sv = s[r][n];
                const float w = live ? fmaf(sv, fmaf(sv, sc.s2, sc.s1), 1.0f) : 0.f;
                den[r] += w;
                sm.w[ty * 4 + r][tx + 8 * n] = w;
            }
        __syncthreads();
#pragma unroll 4
        for (int j = 0; j < kT; ++j) {
            float ww[4], vv[NC];
#pragma unroll
            for (int r = 0; r < 4; ++r) ww[r] = sm.w[ty * 4 + r][j];
#pragma unroll
            for (int c = 0; c < NC; ++c) vv[c] = sm.v[j][tx + 8 * c];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < NC; ++c) num[r][c] = fmaf(ww[r], vv[c], num[r][c]);
        }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        den[r] += __shfl_xor_sync(0xffffffffu, den[r], 1);
        den[r] += __shfl_xor_sync(0xffffffffu, den[r], 2);
        den[r] += __shfl_xor_sync(0xffffffffu, den[r], 4);
    }
    // contribution of a given initial state: phi(q_i).S0 and phi(q_i).z0
    if (kv0 != nullptr) {
        const float* S0 = kv0 + head * (size_t)D * DV;
        const float* Z0 = z0 + head * (size_t)D;
        for (int f = 0; f < D; ++f) {
            float pf[4], srow[NC];
#pragma unroll
            for (int r = 0; r < 4; ++r) pf[r] = phi_gen(sm.q[ty * 4 + r], df, f, sc);
#pragma unroll
            for (int c = 0; c < NC; ++c) srow[c] = S0[(size_t)f * DV + tx + 8 * c];
            const float zf = Z0[f];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                den[r] = fmaf(pf[r], zf, den[r]);
#pragma unroll
                for (int c = 0; c < NC; ++c) num[r][c] = fmaf(pf[r], srow[c], num[r][c]);
            }
        }
    }
    T* oh = out + head * (size_t)L * DV;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int i = i0 + ty * 4 + r;
        if (i >= L) continue;
        const float inv = numerator_only ? 1.0f : 1.0f / (den[r] + kEps);
#pragma unroll
        for (int c = 0; c < NC; ++c) oh[(size_t)i * DV + tx + 8 * c] = from_f32<T>(num[r][c] * inv);
    }
}

// S[f, :] = S0[f, :] + sum_j phi_f(k_j) v_j, z[f] likewise; one CTA per (32 features, head), one thread per
// value column plus one for z (thread DV).  Per block of 32 tokens the 32 x 32 feature values are
// expanded once into shared memory by all threads, then every column thread accumulates from there.
template <typename T, int DV>
__global__ void __launch_bounds__(DV + 32) generic_state_kernel(const T* __restrict__ k, const T* __restrict__ v,
                                                                float* __restrict__ kv, float* __restrict__ z, int L,
                                                                int df, int accumulate) {
    constexpr int FB = 32, TOK = 32, NT = DV + 32;
    __shared__ float s_k[TOK][kMaxDF + 1];
    __shared__ float s_v[TOK][DV];
    __shared__ __align__(16) float s_phi[TOK][FB];
    __shared__ int s_m[FB], s_n[FB];                 // feature -> (m, n) of the product, or (-1, -1) constant, (m, -1) linear
    __shared__ float s_scale[FB];
    const int f0 = blockIdx.x * FB;
    const size_t head = blockIdx.y;
    const int D = expanded_dim(df);
    const FeatScale sc = feat_scale(df);
    const int c = threadIdx.x;                       // value column, or DV for the K-state
    const bool active = c <= DV;
    if (threadIdx.x < FB) {
        const int f = f0 + threadIdx.x;
        int m = -1, n = -1;
        float scale = f < D ? 1.0f : 0.0f;           // rows past the end contribute nothing
        if (f >= 1 && f <= df) { m = f - 1; scale = sc.lin; }
        else if (f > df && f < D) { m = (f - 1 - df) / df; n = (f - 1 - df) % df; scale = sc.quad; }
        s_m[threadIdx.x] = m; s_n[threadIdx.x] = n; s_scale[threadIdx.x] = scale;
    }
    float acc[FB];
#pragma unroll
    for (int r = 0; r < FB; ++r) acc[r] = 0.f;
    const T* kh = k + head * (size_t)L * df;
    const T* vh = v + head * (size_t)L * DV;
    for (int t0 = 0; t0 < L; t0 += TOK) {
        __syncthreads();
        for (int i = threadIdx.x; i < TOK * df; i += NT) {
            const int t = i / df, m = i - t * df;
            s_k[t][m] = t0 + t < L ? to_f32(kh[(size_t)(t0 + t) * df + m]) : 0.f;
        }
        for (int i = threadIdx.x; i < TOK * DV; i += NT) {
            const int t = i / DV, cc = i - t * DV;
            s_v[t][cc] = t0 + t < L ? to_f32(vh[(size_t)(t0 + t) * DV + cc]) : 0.f;
        }
        __syncthreads();
        for (int i = threadIdx.x; i < TOK * FB; i += NT) {
            const int t = i / FB, r = i - t * FB;
            const int m = s_m[r], n = s_n[r];
            float x = s_scale[r];
            if (m >= 0) x *= s_k[t][m];
            if (n >= 0) x *= s_k[t][n];
            s_phi[t][r] = t0 + t < L ? x : 0.f;      // tokens past the end: also no constant feature
        }
        __syncthreads();
        if (active) {
#pragma unroll 4
            for (int t = 0; t < TOK; ++t) {
                const float vc = c < DV ? s_v[t][c] : 1.0f;
#pragma unroll
                for (int r4 = 0; r4 < FB / 4; ++r4) {
                    const float4 p = *reinterpret_cast<const float4*>(&s_phi[t][r4 * 4]);
                    acc[r4 * 4 + 0] = fmaf(p.x, vc, acc[r4 * 4 + 0]);
                    acc[r4 * 4 + 1] = fmaf(p.y, vc, acc[r4 * 4 + 1]);
                    acc[r4 * 4 + 2] = fmaf(p.z, vc, acc[r4 * 4 + 2]);
                    acc[r4 * 4 + 3] = fmaf(p.w, vc, acc[r4 * 4 + 3]);
                }
            }
        }
    }
    if (active) {
#pragma unroll
        for (int r = 0; r < FB; ++r) {
            const int f = f0 + r;
            if (f >= D) continue;
            float* dst = c < DV ? &kv[(head * D + f) * DV + c] : &z[head * D + f];
            *dst = accumulate ? *dst + acc[r] : acc[r];
        }
    }
}

// one recurrent step on the [D, d_v] state of a head (update, then read): the d' = 16 decode kernel's
// stream with the number of rows as a parameter.  d_v / 4 consecutive threads cover a state row with one
// 128-bit load each, six rows are in flight per thread; STREAM: the state of all heads is larger than L2,
// so every line is used once per step and takes the evict-first policy.
template <typename T, int DV, bool STREAM>
__global__ void __launch_bounds__(256, 4) generic_decode_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                                const T* __restrict__ v, float* __restrict__ kv,
                                                                float* __restrict__ z, T* __restrict__ out, int df,
                                                                int numerator_only) {
    constexpr int TPR = DV / 4;                        // threads per state row
    constexpr int RPP = 256 / TPR;                     // rows per pass: 8 (d_v 128), 9 (112), 16 (64)
    constexpr int UNROLL = 6;
    __shared__ float s_x[2][kMaxDF];
    __shared__ float s_pq[1 + kMaxDF + kMaxDF * kMaxDF], s_pk[1 + kMaxDF + kMaxDF * kMaxDF];
    __shared__ __align__(16) float s_num[RPP][DV];     // written with 16-byte stores
    __shared__ float s_den[8];
    const int tid = threadIdx.x;
    const size_t head = blockIdx.x;
    const int D = expanded_dim(df);
    const FeatScale sc = feat_scale(df);
    const int c4 = tid % TPR, rslot = tid / TPR;
    const bool row_thread = rslot < RPP;               // false only for the idle tail threads of d_v 112
    if (tid < df) s_x[0][tid] = to_f32(q[head * df + tid]);
    else if (tid >= 32 && tid < 32 + df) s_x[1][tid - 32] = to_f32(k[head * df + tid - 32]);
    float vv[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) vv[e] = to_f32(v[head * DV + c4 * 4 + e]);
    __syncthreads();
    for (int f = tid; f < D; f += 256) {
        s_pq[f] = phi_gen(s_x[0], df, f, sc);
        s_pk[f] = phi_gen(s_x[1], df, f, sc);
    }
    __syncthreads();
    float dpart = 0.f;
    float* zh = z + head * (size_t)D;
    for (int f = tid; f < D; f += 256) {
        const float zn = zh[f] + s_pk[f];
        zh[f] = zn;
        dpart = fmaf(s_pq[f], zn, dpart);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dpart += __shfl_xor_sync(0xffffffffu, dpart, o);
    if ((tid & 31) == 0) s_den[tid >> 5] = dpart;

    float4* S = reinterpret_cast<float4*>(kv + head * (size_t)D * DV) + c4;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const int npass = (D + RPP - 1) / RPP;
    for (int p0 = 0; p0 < npass; p0 += UNROLL) {
        float4 s[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int r = (p0 + u) * RPP + rslot;
            if (r < D && row_thread) s[u] = STREAM ? __ldcs(&S[(size_t)r * TPR]) : S[(size_t)r * TPR];
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int r = (p0 + u) * RPP + rslot;
            if (r < D && row_thread) {
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
        float num = 0.f, den = 0.f;
#pragma unroll
        for (int r = 0; r < RPP; ++r) num += s_num[r][tid];
#pragma unroll
        for (int w = 0; w < 8; ++w) den += s_den[w];
        out[head * DV + tid] = from_f32<T>(numerator_only ? num : num / (den + kEps));
    }
}

template <typename T, int DV>
static based_status prefill_t(const void* q, const void* k, const void* v, void* out, float* kv, float* z, int BH,
                              int L, int df, int flags, bool outputs_done, cudaStream_t stream) {
    const size_t smem = sizeof(FwdSmem<DV>);
    {
        static bool configured[64] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BASED_ERR_CUDA;
        std::lock_guard<std::mutex> lock(setup_mutex());
        if (!configured[dev]) {
            if (cudaFuncSetAttribute(generic_prefill_kernel<T, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)smem) != cudaSuccess)
                return BASED_ERR_CUDA;
            configured[dev] = true;
        }
    }
    const bool cont = (flags & BASED_STATE_CONTINUE) != 0;
    const T* qq = static_cast<const T*>(q);
    const T* kk = static_cast<const T*>(k);
    const T* vv = static_cast<const T*>(v);
    based_status st = BASED_OK;
    if (!outputs_done) {
        generic_prefill_kernel<T, DV><<<dim3((L + kT - 1) / kT, BH), kBT, smem, stream>>>(
            qq, kk, vv, static_cast<T*>(out), cont ? kv : nullptr, cont ? z : nullptr, L, df,
            (flags & BASED_NUMERATOR_ONLY) ? 1 : 0);
        note_launch();
        st = check_launch("generic_prefill_kernel");
    }
    if (st != BASED_OK || kv == nullptr) return st;
    if (sizeof(T) == 2) return launch_state_generic_tc(k, v, kv, z, BH, L, df, DV, cont ? 1 : 0, stream);
    const int D = expanded_dim(df);
    generic_state_kernel<T, DV><<<dim3((D + 31) / 32, BH), DV + 32, 0, stream>>>(kk, vv, kv, z, L, df, cont ? 1 : 0);
    note_launch();
    return check_launch("generic_state_kernel");
}

based_status launch_prefill_generic(const void* q, const void* k, const void* v, void* out, float* kv, float* z,
                                    int BH, int L, int d_feat, int d_v, based_dtype io, int flags, bool outputs_done,
                                    cudaStream_t stream) {
    if (io == BASED_F32) {
        if (d_v == 64) return prefill_t<float, 64>(q, k, v, out, kv, z, BH, L, d_feat, flags, outputs_done, stream);
        if (d_v == 112) return prefill_t<float, 112>(q, k, v, out, kv, z, BH, L, d_feat, flags, outputs_done, stream);
        return prefill_t<float, 128>(q, k, v, out, kv, z, BH, L, d_feat, flags, outputs_done, stream);
    }
    if (d_v == 64) return prefill_t<__nv_bfloat16, 64>(q, k, v, out, kv, z, BH, L, d_feat, flags, outputs_done, stream);
    if (d_v == 112) return prefill_t<__nv_bfloat16, 112>(q, k, v, out, kv, z, BH, L, d_feat, flags, outputs_done, stream);
    return prefill_t<__nv_bfloat16, 128>(q, k, v, out, kv, z, BH, L, d_feat, flags, outputs_done, stream);
}

// The state of a token block alone, any supported feature dimension (16 included): bf16 io on tensor cores,
// fp32 io with fp32 FMAs.
template <int DV>
static based_status state_f32(const void* k, const void* v, float* kv, float* z, int BH, int L, int df, int cont,
                              cudaStream_t stream) {
    const int D = expanded_dim(df);
    generic_state_kernel<float, DV><<<dim3((D + 31) / 32, BH), DV + 32, 0, stream>>>(
        static_cast<const float*>(k), static_cast<const float*>(v), kv, z, L, df, cont);
    note_launch();
    return check_launch("generic_state_kernel");
}

based_status launch_state_generic(const void* k, const void* v, float* kv, float* z, int BH, int L, int d_feat, int d_v,
                                  based_dtype io, int cont, cudaStream_t stream) {
    if (io == BASED_BF16) return launch_state_generic_tc(k, v, kv, z, BH, L, d_feat, d_v, cont, stream);
    if (d_v == 64) return state_f32<64>(k, v, kv, z, BH, L, d_feat, cont, stream);
    if (d_v == 112) return state_f32<112>(k, v, kv, z, BH, L, d_feat, cont, stream);
    return state_f32<128>(k, v, kv, z, BH, L, d_feat, cont, stream);
}

template <typename T, int DV>
static based_status decode_t(const void* q, const void* k, const void* v, float* kv, float* z, void* out, int BH,
                             int df, int num_only, cudaStream_t stream) {
    // 96 MB: safely above what L2 (126 MB, shared with everything else) keeps from one step to the next
    const bool streaming = (size_t)BH * expanded_dim(df) * DV * sizeof(float) > (size_t)96 << 20;
    const T* qq = static_cast<const T*>(q);
    const T* kk = static_cast<const T*>(k);
    const T* vv = static_cast<const T*>(v);
    if (streaming) generic_decode_kernel<T, DV, true><<<BH, 256, 0, stream>>>(qq, kk, vv, kv, z, static_cast<T*>(out), df, num_only);
    else generic_decode_kernel<T, DV, false><<<BH, 256, 0, stream>>>(qq, kk, vv, kv, z, static_cast<T*>(out), df, num_only);
    note_launch();
    return check_launch("generic_decode_kernel");
}

template <typename T>
static based_status decode_dv(const void* q, const void* k, const void* v, float* kv, float* z, void* out, int BH,
                              int df, int d_v, int num_only, cudaStream_t stream) {
    if (d_v == 64) return decode_t<T, 64>(q, k, v, kv, z, out, BH, df, num_only, stream);
    if (d_v == 112) return decode_t<T, 112>(q, k, v, kv, z, out, BH, df, num_only, stream);
    return decode_t<T, 128>(q, k, v, kv, z, out, BH, df, num_only, stream);
}

based_status launch_decode_generic(const void* q, const void* k, const void* v, float* kv, float* z, void* out,
                                   int BH, int d_feat, int d_v, based_dtype io, bool numerator_only,
                                   cudaStream_t stream) {
    if (io == BASED_F32) return decode_dv<float>(q, k, v, kv, z, out, BH, d_feat, d_v, numerator_only ? 1 : 0, stream);
    return decode_dv<__nv_bfloat16>(q, k, v, kv, z, out, BH, d_feat, d_v, numerator_only ? 1 : 0, stream);
}

}  // namespace based
