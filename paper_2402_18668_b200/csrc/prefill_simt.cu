// based_prefill, fp32 SIMT path: causal Taylor linear attention evaluated in its
// recurrent form (Sec. 4.1 recurrences) with the whole [273, d_v] state of a head
// held in registers, fp32 FMAs only.  This is the path for fp32 inputs, whose
// 1e-4 tolerance tensor-core operand formats (bf16, tf32) cannot meet.
//
// One CTA per (b, h).  Thread (g, c) owns column c of the state for the feature
// rows of group g (4 groups of 72 padded rows); an extra warp carries the "ones
// column", i.e. the K-state z, so numerator and denominator run the same code.
// Tokens are processed in batches of 8: their features are expanded once into
// shared memory, then every thread does  S += phi(k) v ;  acc += phi(q) S  per
// token; partial sums of the 4 groups are combined through shared memory.
#include "common.cuh"

namespace based {

namespace {
constexpr int kGroups = 4;
constexpr int kRowsPerGroup = 72;                    // 4 * 72 = 288 >= 273, zero padded
constexpr int kDPad = kGroups * kRowsPerGroup;
constexpr int kTok = 8;                              // tokens per batch
}  // namespace

template <int DV, typename T>
__global__ void __launch_bounds__(kGroups* DV + 32, 1)
    prefill_simt_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                        T* __restrict__ out, float* __restrict__ kv, float* __restrict__ z, int L, int flags) {
    constexpr int NT = kGroups * DV + 32;
    __shared__ __align__(16) float s_pq[kTok][kDPad];
    __shared__ __align__(16) float s_pk[kTok][kDPad];
    __shared__ float s_x[2][kTok][kDFeat];
    __shared__ float s_v[kTok][DV];
    __shared__ float s_part[kGroups][kTok][DV + 1];

    const int tid = threadIdx.x;
    const size_t head = blockIdx.x;
    const bool ones = tid >= kGroups * DV;           // the warp that carries z
    const int g = ones ? (tid - kGroups * DV) : tid / DV;
    const int c = ones ? DV : tid % DV;
    const bool active = !ones || g < kGroups;

    float S[kRowsPerGroup];
#pragma unroll
    for (int j = 0; j < kRowsPerGroup; ++j) S[j] = 0.f;
    // Symmetric state format: full row (m, n) lives in symmetric row (min, max), scaled by sqrt 2
    // off the diagonal.  Rows (m, n) and (n, m) of the full state are bitwise equal here (same
    // products, same order of accumulation), so the fold (S_mn + S_nm) / sqrt 2 is S_mn * sqrt 2.
    const bool sym = (flags & BASED_STATE_SYM) != 0;
    const int nrows = sym ? kDSym : kD;
    auto sym_row = [](int p, float& scale, bool& owner) -> int {
        scale = 1.f;
        owner = true;
        if (p <= kDFeat) return p;
        const int m = (p - 1 - kDFeat) >> 4, n = (p - 1 - kDFeat) & 15;
        owner = m <= n;
        if (m != n) scale = 0.70710678118654752f;
        return m <= n ? sym_pair_row(m, n) : sym_pair_row(n, m);
    };
    if (active && (flags & BASED_STATE_CONTINUE)) {
#pragma unroll
        for (int j = 0; j < kRowsPerGroup; ++j) {
            const int p = g * kRowsPerGroup + j;
            if (p < kD) {
                float scale = 1.f;
                bool owner;
                const int r = sym ? sym_row(p, scale, owner) : p;
                S[j] = (ones ? z[head * nrows + r] : kv[(head * nrows + r) * DV + c]) * scale;
            }
        }
    }

    const T* qh = q + head * (size_t)L * kDFeat;
    const T* kh = k + head * (size_t)L * kDFeat;
    const T* vh = v + head * (size_t)L * DV;
    T* oh = out + head * (size_t)L * DV;

    for (int t0 = 0; t0 < L; t0 += kTok) {
        const int nt = min(kTok, L - t0);
        for (int i = tid; i < kTok * kDFeat; i += NT) {
            const int t = i / kDFeat;
            s_x[0][t][i % kDFeat] = t < nt ? to_f32(qh[(size_t)t0 * kDFeat + i]) : 0.f;
            s_x[1][t][i % kDFeat] = t < nt ? to_f32(kh[(size_t)t0 * kDFeat + i]) : 0.f;
        }
        for (int i = tid; i < kTok * DV; i += NT) {
            const int t = i / DV;
            s_v[t][i % DV] = t < nt ? to_f32(vh[(size_t)t0 * DV + i]) : 0.f;
        }
        __syncthreads();
        for (int i = tid; i < kTok * kDPad; i += NT) {
            const int t = i / kDPad, p = i % kDPad;
            const bool live = p < kD && t < nt;      // padded rows and tokens past the end contribute nothing
            s_pq[t][p] = live ? phi_at(s_x[0][t], p) : 0.f;
            s_pk[t][p] = live ? phi_at(s_x[1][t], p) : 0.f;
        }
        __syncthreads();
        if (active) {
#pragma unroll
            for (int t = 0; t < kTok; ++t) {
                const float vc = ones ? 1.f : s_v[t][c];
                const float4* pk4 = reinterpret_cast<const float4*>(&s_pk[t][g * kRowsPerGroup]);
                const float4* pq4 = reinterpret_cast<const float4*>(&s_pq[t][g * kRowsPerGroup]);
                float a = 0.f;
#pragma unroll
                for (int j4 = 0; j4 < kRowsPerGroup / 4; ++j4) {
                    const float4 fk = pk4[j4], fq = pq4[j4];
                    S[4 * j4 + 0] = fmaf(fk.x, vc, S[4 * j4 + 0]);
                    S[4 * j4 + 1] = fmaf(fk.y, vc, S[4 * j4 + 1]);
                    S[4 * j4 + 2] = fmaf(fk.z, vc, S[4 * j4 + 2]);
                    S[4 * j4 + 3] = fmaf(fk.w, vc, S[4 * j4 + 3]);
                    a = fmaf(fq.x, S[4 * j4 + 0], a);
                    a = fmaf(fq.y, S[4 * j4 + 1], a);
                    a = fmaf(fq.z, S[4 * j4 + 2], a);
                    a = fmaf(fq.w, S[4 * j4 + 3], a);
                }
                s_part[g][t][c] = a;
            }
        }
        __syncthreads();
        for (int i = tid; i < nt * DV; i += NT) {
            const int t = i / DV, cc = i % DV;
            float num = 0.f, den = 0.f;
#pragma unroll
            for (int gg = 0; gg < kGroups; ++gg) {
                num += s_part[gg][t][cc];
                den += s_part[gg][t][DV];
            }
            oh[(size_t)t0 * DV + i] = from_f32<T>((flags & BASED_NUMERATOR_ONLY) ? num : num / (den + kEps));
        }
    }

    if (kv != nullptr && active) {
#pragma unroll
        for (int j = 0; j < kRowsPerGroup; ++j) {
            const int p = g * kRowsPerGroup + j;
            if (p < kD) {
                float scale = 1.f;
                bool owner = true;
                const int r = sym ? sym_row(p, scale, owner) : p;
                if (!owner) continue;                       // the (n, m) twin writes the shared row
                const float val = sym && scale != 1.f ? S[j] * 1.41421356237309505f : S[j];
                if (ones) z[head * nrows + r] = val;
                else kv[(head * nrows + r) * DV + c] = val;
            }
        }
    }
}

template <int DV, typename T>
static based_status launch_t(const void* q, const void* k, const void* v, void* out, float* kv, float* z, int BH,
                             int L, int flags, cudaStream_t stream) {
    prefill_simt_kernel<DV, T><<<BH, kGroups * DV + 32, 0, stream>>>(
        static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), static_cast<T*>(out), kv, z,
        L, flags);
    note_launch();
    return check_launch("prefill_simt_kernel");
}

based_status launch_prefill_simt(const void* q, const void* k, const void* v, void* out, float* kv, float* z,
                                 int BH, int L, int d_v, based_dtype io, int flags, cudaStream_t stream) {
    if (d_v == 64) {
        return io == BASED_F32 ? launch_t<64, float>(q, k, v, out, kv, z, BH, L, flags, stream)
                               : launch_t<64, __nv_bfloat16>(q, k, v, out, kv, z, BH, L, flags, stream);
    }
    if (d_v == 112) {
        return io == BASED_F32 ? launch_t<112, float>(q, k, v, out, kv, z, BH, L, flags, stream)
                               : launch_t<112, __nv_bfloat16>(q, k, v, out, kv, z, BH, L, flags, stream);
    }
    return io == BASED_F32 ? launch_t<128, float>(q, k, v, out, kv, z, BH, L, flags, stream)
                           : launch_t<128, __nv_bfloat16>(q, k, v, out, kv, z, BH, L, flags, stream);
}

}  // namespace based
