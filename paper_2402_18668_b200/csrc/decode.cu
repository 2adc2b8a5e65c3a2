// based_decode_step: one recurrent step of Taylor linear attention per (b, h).
//
// Computes the KV-state / K-state recurrences of Sec. 4.1 in the update-then-read
// order of the App. B.2 step() listing:  S += phi(k) v^T,  z += phi(k),
// y = phi(q) S / (phi(q).z + eps).  Unlike Algorithm 2, q and k arrive raw (16 wide)
// and the 273 features are expanded on chip.
//
// The step is a pure stream over the fp32 state: each head's [273, d_v] block is
// read once and written once (2 * 273 * d_v * 4 bytes per head), 0.5 flop per byte,
// so the kernel is bounded by HBM bandwidth.  One CTA of 256 threads owns one head.
// A state row is covered by d_v/4 consecutive threads with one 128-bit load each, so
// every warp instruction touches whole 512-byte (d_v=128) or two 256-byte (d_v=64)
// rows; loads of several rows are issued before the first dependent FMA to keep
// many bytes in flight per SM (4 CTAs per SM).
#include "common.cuh"
#include "decode.cuh"

namespace based {

template <int DV, typename T, bool STREAM, bool SYM>
__global__ void __launch_bounds__(256, 4) decode_step_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                          const T* __restrict__ v, float* __restrict__ kv,
                                                          float* __restrict__ z, T* __restrict__ out,
                                                          int numerator_only) {
    decode_step_body<DV, T, STREAM, SYM>(q, k, v, kv, z, out, numerator_only, blockIdx.x);
}

template <int DV, typename T, bool SYM>
static based_status launch_t(const void* q, const void* k, const void* v, float* kv, float* z, void* out, int BH,
                             int num_only, cudaStream_t stream) {
    // 96 MB: safely above what L2 (126 MB, shared with everything else) keeps from one step to the next
    const bool streaming = (size_t)BH * (SYM ? kDSym : kD) * DV * sizeof(float) > (size_t)96 << 20;
    if (streaming)
        decode_step_kernel<DV, T, true, SYM><<<BH, 256, 0, stream>>>(
            static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), kv, z, static_cast<T*>(out),
            num_only);
    else
        decode_step_kernel<DV, T, false, SYM><<<BH, 256, 0, stream>>>(
            static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), kv, z, static_cast<T*>(out),
            num_only);
    note_launch();
    return check_launch("decode_step_kernel");
}

template <int DV, bool SYM>
static based_status launch_dv(const void* q, const void* k, const void* v, float* kv, float* z, void* out, int BH,
                              based_dtype io, int num_only, cudaStream_t stream) {
    return io == BASED_F32 ? launch_t<DV, float, SYM>(q, k, v, kv, z, out, BH, num_only, stream)
                           : launch_t<DV, __nv_bfloat16, SYM>(q, k, v, kv, z, out, BH, num_only, stream);
}

based_status launch_decode(const void* q, const void* k, const void* v, float* kv, float* z, void* out, int BH,
                           int d_v, based_dtype io, bool sym, bool numerator_only, cudaStream_t stream) {
    const int n = numerator_only ? 1 : 0;
    if (d_v == 64)
        return sym ? launch_dv<64, true>(q, k, v, kv, z, out, BH, io, n, stream)
                   : launch_dv<64, false>(q, k, v, kv, z, out, BH, io, n, stream);
    if (d_v == 112)
        return sym ? launch_dv<112, true>(q, k, v, kv, z, out, BH, io, n, stream)
                   : launch_dv<112, false>(q, k, v, kv, z, out, BH, io, n, stream);
    return sym ? launch_dv<128, true>(q, k, v, kv, z, out, BH, io, n, stream)
               : launch_dv<128, false>(q, k, v, kv, z, out, BH, io, n, stream);
}

// ------------------------------------------------------------------ full <-> symmetric state
// One CTA per head.  to_sym: row (m,n), m < n, becomes (S_mn + S_nm) / sqrt 2, the other rows are
// copied; from_sym: rows (m,n) and (n,m) both become S_sym / sqrt 2 (a full state that gives the
// same outputs; a state built by the recurrences is symmetric, so this is its inverse).
__global__ void __launch_bounds__(256) state_convert_kernel(const float* __restrict__ kv_in,
                                                            const float* __restrict__ z_in,
                                                            float* __restrict__ kv_out, float* __restrict__ z_out,
                                                            int d_v, bool to_sym) {
    constexpr float kRs2 = 0.70710678118654752f;
    const size_t head = blockIdx.x;
    const int nin = to_sym ? kD : kDSym, nout = to_sym ? kDSym : kD;
    const float* kvi = kv_in + head * (size_t)nin * d_v;
    const float* zi = z_in + head * (size_t)nin;
    float* kvo = kv_out + head * (size_t)nout * d_v;
    float* zo = z_out + head * (size_t)nout;
    // source rows of output row r: (a, b >= 0 -> (a + b) scaled, b < 0 -> copy of a, scaled for from_sym pairs)
    auto src = [&](int r, int& a, int& b, float& scale) {
        b = -1;
        scale = 1.f;
        if (r <= kDFeat) { a = r; return; }
        if (to_sym) {
            int m, n;
            pair_of(r - 1 - kDFeat, m, n);
            a = 1 + kDFeat + m * kDFeat + n;
            if (m != n) { b = 1 + kDFeat + n * kDFeat + m; scale = kRs2; }
        } else {
            const int p = r - 1 - kDFeat;
            int m = p >> 4, n = p & 15;
            if (m > n) { const int t = m; m = n; n = t; }
            a = 1 + kDFeat + m * kDFeat - m * (m - 1) / 2 + (n - m);
            if (m != n) scale = kRs2;
        }
    };
    // d_v / 4 consecutive threads cover a row with one 128-bit access each (d_v 112: 28 threads per row, 9 rows per pass)
    const int tpr = d_v >> 2, rpp = blockDim.x / tpr;
    const int c4 = threadIdx.x % tpr, rslot = threadIdx.x / tpr;
    if (rslot < rpp) {
        for (int r = rslot; r < nout; r += rpp) {
            int a, b;
            float scale;
            src(r, a, b, scale);
            float4 x = __ldcs(reinterpret_cast<const float4*>(kvi + (size_t)a * d_v) + c4);
            if (b >= 0) {
                const float4 y = __ldcs(reinterpret_cast<const float4*>(kvi + (size_t)b * d_v) + c4);
                x.x += y.x; x.y += y.y; x.z += y.z; x.w += y.w;
            }
            x.x *= scale; x.y *= scale; x.z *= scale; x.w *= scale;
            __stcs(reinterpret_cast<float4*>(kvo + (size_t)r * d_v) + c4, x);
        }
    }
    for (int r = threadIdx.x; r < nout; r += blockDim.x) {
        int a, b;
        float scale;
        src(r, a, b, scale);
        float x = zi[a];
        if (b >= 0) x += zi[b];
        zo[r] = x * scale;
    }
}

namespace {
template <typename K>
bool load_kernel(K kernel) {
    cudaFuncAttributes attr;
    return cudaFuncGetAttributes(&attr, kernel) == cudaSuccess;
}
template <int DV, typename T>
bool load_decode_variants() {
    return load_kernel(decode_step_kernel<DV, T, false, false>) && load_kernel(decode_step_kernel<DV, T, true, false>) &&
           load_kernel(decode_step_kernel<DV, T, false, true>) && load_kernel(decode_step_kernel<DV, T, true, true>);
}
}  // namespace

// Forces the decode kernels into the current context (first use inside a stream capture would
// otherwise load them there).
based_status preload_decode() {
    const bool ok = load_decode_variants<64, float>() && load_decode_variants<64, __nv_bfloat16>() &&
                    load_decode_variants<112, float>() && load_decode_variants<112, __nv_bfloat16>() &&
                    load_decode_variants<128, float>() && load_decode_variants<128, __nv_bfloat16>() &&
                    load_kernel(state_convert_kernel);
    return ok ? BASED_OK : BASED_ERR_CUDA;
}

based_status launch_state_convert(const float* kv_in, const float* z_in, float* kv_out, float* z_out, int BH,
                                  int d_v, bool to_sym, cudaStream_t stream) {
    state_convert_kernel<<<BH, 256, 0, stream>>>(kv_in, z_in, kv_out, z_out, d_v, to_sym);
    note_launch();
    return check_launch("state_convert_kernel");
}

}  // namespace based
