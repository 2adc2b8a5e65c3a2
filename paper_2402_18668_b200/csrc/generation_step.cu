// based_generation_step: one generated token through both mixers of a Based layer pair in ONE launch.
//
// The linear-attention decode step (Sec. 4.1 recurrences, Algorithm 2) streams each head's fp32 state once;
// the sliding-window decode step (Algorithm 3) reads a small rolling cache.  The paper runs next-token
// prediction under CUDA graphs (Sec. 6, "Efficiency Benchmarks") because at these sizes launch and fill
// latencies are a visible share of a step.  As two kernels, even as two branches of one graph, the short
// window step runs after (or before) the long state stream: the state kernel's CTAs fill every SM's
// register file, so the other kernel's CTAs wait for a wave to drain.  Here both kinds of CTA are one
// grid, dealt out in turn (one window CTA, holding two heads, per two state CTAs), so the window heads'
// bulk copies and their fill and drain latency ride in the shadow of the state stream and the step costs
// one launch.
//
// CTA roles by block index (256 threads each):
//   window role: two groups of 128 threads, one head each, the code of swa_decode_kernel with a named
//                barrier per group (swa_decode.cuh);
//   state role:  the code of decode_step_kernel (decode.cuh).
#include "decode.cuh"
#include "swa_decode.cuh"

namespace based {

namespace {
using namespace swa_dec;

struct GenArgs {
    // linear attention
    const void *q, *k, *v;
    float *kv, *z;
    void* out;
    int n_lin;            // heads
    int numerator_only;
    // sliding window
    const void *qw, *kw, *vw;
    void *kc, *vc, *outw;
    int n_swa;            // heads
    int window;
    int* pos_state;       // {position, ticket}
    float scale;
    unsigned int* err;
    // dealing of the roles
    int n_pairs;          // leading triples (window CTA, state CTA, state CTA)
    int swa_group_bytes;  // shared memory of one 128-thread window group
};

template <int DV, typename T, bool STREAM, bool SYM, int NPW>
__global__ void __launch_bounds__(256, 4) generation_step_kernel(const GenArgs a) {
    extern __shared__ __align__(128) unsigned char smem[];
    // block index -> role: the first 3 * n_pairs blocks come in triples (window, state, state); then
    // whatever window CTAs are left, then the remaining state CTAs
    const int i = blockIdx.x, n_swa_ctas = (a.n_swa + 1) / 2;
    int swa_cta = -1, lin_head = -1;
    if (i < 3 * a.n_pairs) {
        const int g = i / 3, r = i - 3 * g;
        if (r == 0) swa_cta = g;
        else lin_head = 2 * g + r - 1;
    } else {
        const int j = i - 3 * a.n_pairs;
        if (j < n_swa_ctas - a.n_pairs) swa_cta = a.n_pairs + j;
        else lin_head = 2 * a.n_pairs + j - (n_swa_ctas - a.n_pairs);
    }
    if (swa_cta >= 0) {
        const int half = threadIdx.x >> 7;
        const int head = 2 * swa_cta + half;
        if (head < a.n_swa) {
            const T* qw = static_cast<const T*>(a.qw);
            const T* kw = static_cast<const T*>(a.kw);
            const T* vw = static_cast<const T*>(a.vw);
            T* kc = static_cast<T*>(a.kc);
            T* vc = static_cast<T*>(a.vc);
            T* ow = static_cast<T*>(a.outw);
            // one named barrier per group (a compile-time id keeps the CTA's barrier count at three)
            if (half == 0)
                swa_decode_body<T, NPW, 1>(qw, kw, vw, kc, vc, ow, a.window, 0, a.pos_state, a.pos_state, a.scale, a.err,
                                           (size_t)head, threadIdx.x & 127, a.n_swa, smem);
            else
                swa_decode_body<T, NPW, 2>(qw, kw, vw, kc, vc, ow, a.window, 0, a.pos_state, a.pos_state, a.scale, a.err,
                                           (size_t)head, threadIdx.x & 127, a.n_swa, smem + a.swa_group_bytes);
        }
    } else {
        decode_step_body<DV, T, STREAM, SYM>(static_cast<const T*>(a.q), static_cast<const T*>(a.k),
                                             static_cast<const T*>(a.v), a.kv, a.z, static_cast<T*>(a.out),
                                             a.numerator_only, (size_t)lin_head);
    }
}

template <int DV, typename T, bool STREAM, bool SYM, int NPW>
based_status launch_k(const GenArgs& a, size_t smem, cudaStream_t stream) {
    auto kern = generation_step_kernel<DV, T, STREAM, SYM, NPW>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return BASED_ERR_CUDA;
    const int grid = a.n_lin + (a.n_swa + 1) / 2;
    kern<<<grid, 256, smem, stream>>>(a);
    note_launch();
    return check_launch("generation_step_kernel");
}

template <int DV, typename T, bool STREAM, bool SYM>
based_status launch_w(const GenArgs& a, size_t smem, cudaStream_t stream) {
    return a.window <= 64 ? launch_k<DV, T, STREAM, SYM, 4>(a, smem, stream) : launch_k<DV, T, STREAM, SYM, 8>(a, smem, stream);
}
template <int DV, typename T>
based_status launch_s(const GenArgs& a, size_t smem, bool sym, bool streaming, cudaStream_t stream) {
    if (sym) return streaming ? launch_w<DV, T, true, true>(a, smem, stream) : launch_w<DV, T, false, true>(a, smem, stream);
    return streaming ? launch_w<DV, T, true, false>(a, smem, stream) : launch_w<DV, T, false, false>(a, smem, stream);
}
template <typename T>
based_status launch_d(const GenArgs& a, int d_v, bool sym, cudaStream_t stream) {
    const size_t group = (swa_decode_smem_bytes<T>(a.window) + 127) & ~(size_t)127;
    GenArgs b = a;
    b.swa_group_bytes = (int)group;
    const size_t smem = 2 * group;
    // as in the stand-alone decode step: evict-first accesses once the state of all heads outgrows L2
    const bool streaming = (size_t)a.n_lin * (sym ? kDSym : kD) * d_v * sizeof(float) > (size_t)96 << 20;
    if (d_v == 64) return launch_s<64, T>(b, smem, sym, streaming, stream);
    if (d_v == 112) return launch_s<112, T>(b, smem, sym, streaming, stream);
    return launch_s<128, T>(b, smem, sym, streaming, stream);
}
}  // namespace

namespace {
template <int DV, typename T, bool STREAM, bool SYM, int NPW>
bool load_one() {
    auto kern = generation_step_kernel<DV, T, STREAM, SYM, NPW>;
    cudaFuncAttributes attr;
    // the largest request a launch of this variant can make: two groups at the widest window it serves
    const size_t group = (swa_decode_smem_bytes<T>(NPW == 4 ? 64 : 128) + 127) & ~(size_t)127;
    return cudaFuncGetAttributes(&attr, kern) == cudaSuccess &&
           cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(2 * group)) == cudaSuccess;
}
template <int DV, typename T>
bool load_dv() {
    return load_one<DV, T, false, false, 4>() && load_one<DV, T, false, false, 8>() && load_one<DV, T, true, false, 4>() &&
           load_one<DV, T, true, false, 8>() && load_one<DV, T, false, true, 4>() && load_one<DV, T, false, true, 8>() &&
           load_one<DV, T, true, true, 4>() && load_one<DV, T, true, true, 8>();
}
}  // namespace

// Loads every variant into the current context and sets its shared-memory limit, so that a first use
// inside a stream capture does neither.
based_status preload_generation_step() {
    const bool ok = load_dv<64, float>() && load_dv<64, __nv_bfloat16>() && load_dv<112, float>() &&
                    load_dv<112, __nv_bfloat16>() && load_dv<128, float>() && load_dv<128, __nv_bfloat16>();
    return ok ? BASED_OK : BASED_ERR_CUDA;
}

based_status launch_generation_step(const void* q, const void* k, const void* v, float* kv, float* z, void* out,
                                    int n_lin, int d_v, bool sym, bool numerator_only, const void* qw, const void* kw,
                                    const void* vw, void* kc, void* vc, void* outw, int n_swa, int window,
                                    int* pos_state, float scale, based_dtype io, cudaStream_t stream) {
    GenArgs a{};
    a.q = q; a.k = k; a.v = v; a.kv = kv; a.z = z; a.out = out; a.n_lin = n_lin; a.numerator_only = numerator_only ? 1 : 0;
    a.qw = qw; a.kw = kw; a.vw = vw; a.kc = kc; a.vc = vc; a.outw = outw; a.n_swa = n_swa; a.window = window;
    a.pos_state = pos_state; a.scale = scale;
    if (error_word_ptr(&a.err) != BASED_OK) return BASED_ERR_CUDA;
    const int n_swa_ctas = (n_swa + 1) / 2;
    a.n_pairs = n_swa_ctas < n_lin / 2 ? n_swa_ctas : n_lin / 2;
    return io == BASED_F32 ? launch_d<float>(a, d_v, sym, stream) : launch_d<__nv_bfloat16>(a, d_v, sym, stream);
}

}  // namespace based
