// Shared host/device helpers of libbased (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>

#include "based.h"

namespace based {

constexpr int kDFeat = 16;                              // d' of the paper
constexpr int kD = 1 + kDFeat + kDFeat * kDFeat;        // 273 expanded features
constexpr int kDSym = 1 + kDFeat + kDFeat * (kDFeat + 1) / 2;   // 153 features, one per unordered pair
constexpr float kEps = 1e-12f;                          // eps of the paper's listings
// feature-map scales: x / d'^(1/4) and x_m x_n / (sqrt(2) sqrt(d')), d' = 16
constexpr float kLinScale = 0.5f;
constexpr float kQuadScale = 0.17677669529663687f;      // 1 / (4 sqrt 2)

// Device address of the sticky status word of the current device (bit 0: a bounded
// wait timed out).  Kernels that can time out receive it as an argument.
based_status error_word_ptr(unsigned int** ptr);

// serialises the per-device one-time set-up of the launchers (function attributes and the like)
std::mutex& setup_mutex();

// host-side bookkeeping
void note_launch();                                     // ++launch counter
based_status check_launch(const char* what);            // cudaGetLastError -> status

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// value of expanded feature f (0..272) of a raw 16-vector x held in registers/shared memory
__device__ __forceinline__ float phi_at(const float* x, int f) {
    if (f == 0) return 1.0f;
    if (f <= kDFeat) return x[f - 1] * kLinScale;
    const int p = f - 1 - kDFeat;
    return x[p >> 4] * x[p & 15] * kQuadScale;
}

// Symmetric feature set: index 0 the constant, 1..16 the linear terms, then the pairs m <= n in
// row-major order of the upper triangle.  pair_of(p) returns (m, n) of pair p in [0, 136).
__host__ __device__ __forceinline__ void pair_of(int p, int& m, int& n) {
    m = 0;
    while (p >= kDFeat - m) {
        p -= kDFeat - m;
        ++m;
    }
    n = m + p;
}
// row of pair (m, n), m <= n, in the symmetric layout
__host__ __device__ constexpr int sym_pair_row(int m, int n) {
    return 1 + kDFeat + m * kDFeat - m * (m - 1) / 2 + (n - m);
}
// value of symmetric feature f (0..152): x_m^2 / (4 sqrt 2) on the diagonal, x_m x_n / 4 off it
__device__ __forceinline__ float psi_at(const float* x, int f) {
    if (f == 0) return 1.0f;
    if (f <= kDFeat) return x[f - 1] * kLinScale;
    int m, n;
    pair_of(f - 1 - kDFeat, m, n);
    return x[m] * x[n] * (m == n ? kQuadScale : 0.25f);
}

// kernel launchers (defined in the .cu files; all asynchronous on `stream`)
// sym: the state has the 153 symmetric rows instead of the 273 full ones
based_status launch_decode(const void* q, const void* k, const void* v, float* kv, float* z, void* out,
                           int BH, int d_v, based_dtype io, bool sym, bool numerator_only, cudaStream_t stream);
// both mixers' decode steps of one token in one launch (generation_step.cu)
based_status launch_generation_step(const void* q, const void* k, const void* v, float* kv, float* z, void* out,
                                    int n_lin, int d_v, bool sym, bool numerator_only, const void* qw, const void* kw,
                                    const void* vw, void* kc, void* vc, void* outw, int n_swa, int window,
                                    int* pos_state, float scale, based_dtype io, cudaStream_t stream);
based_status preload_generation_step();
// full (273-row) state -> symmetric (153-row) state, or back
based_status launch_state_convert(const float* kv_in, const float* z_in, float* kv_out, float* z_out, int BH,
                                  int d_v, bool to_sym, cudaStream_t stream);
based_status launch_prefill_simt(const void* q, const void* k, const void* v, void* out, float* kv, float* z,
                                 int BH, int L, int d_v, based_dtype io, int flags, cudaStream_t stream);
// bf16 tensor-core prefill (tcgen05); workspace holds partial states of sequence segments.  prefill_tc_workspace_bytes
// is what the fastest plan needs; workspace_limit = the bytes behind `workspace`: a call given less takes the fastest
// plan that fits (fewer segments per head, in the end none: the plain loop and the recompute mode need no workspace).
size_t prefill_tc_workspace_bytes(int BH, int L, int d_v);
based_status launch_prefill_tc(const void* q, const void* k, const void* v, void* out, float* kv, float* z, int BH,
                               int L, int d_v, int flags, void* workspace, cudaStream_t stream,
                               size_t workspace_limit = ~(size_t)0);
// based_prefill without its workspace check: the plan is fitted to the workspace given (for based_prefill_static_scratch)
based_status prefill_fit_workspace(const void* q, const void* k, const void* v, void* out, float* kv_state, float* z_state,
                                   int B, int H, int L, int d_feat, int d_v, based_dtype io, int flags, void* workspace,
                                   size_t workspace_bytes, void* cuda_stream);
// bf16 tensor-core sliding window (window <= 128)
bool swa_tc_supported(int window);
based_status launch_swa_tc(const void* q, const void* k, const void* v, void* out, int BH, int L, int window,
                           float scale, cudaStream_t stream);
// pos_dev != nullptr: the position is read from device memory by the kernel (pos is ignored);
// pos_adv != nullptr ({position, ticket}, pos_dev == pos_adv): the kernel also stores position + 1 at its end
based_status launch_swa_decode(const void* q, const void* k, const void* v, void* kc, void* vc, void* out, int BH,
                               int window, int pos, const int* pos_dev, int* pos_adv, float scale, based_dtype io,
                               cudaStream_t stream, int pos_group = 0);
// gated short convolution (BaseConv core); step: one token on a [B, width-1, C] state, N ignored
based_status launch_baseconv(const void* a, const void* g, const float* h, const float* b2, void* state, void* out,
                             int B, int N, int C, int width, bool step, based_dtype io, cudaStream_t stream);
// backward of the linear attention (fp32 FMA, quadratic form); stats: [BH, L] float2 scratch
based_status launch_prefill_backward(const void* q, const void* k, const void* v, const void* g, void* dq, void* dk,
                                     void* dv, float* stats, int BH, int L, int d_v, based_dtype io,
                                     int numerator_only, cudaStream_t stream);
// feature dimensions 8, 24, 32 (fp32 FMA, definition form); state layout [1 + d' + d'^2, d_v]
// outputs_done: out has been written already (tensor-core forward), only the state is still to do
based_status launch_prefill_generic(const void* q, const void* k, const void* v, void* out, float* kv, float* z,
                                    int BH, int L, int d_feat, int d_v, based_dtype io, int flags, bool outputs_done,
                                    cudaStream_t stream);
// the final state of those feature dimensions on tensor cores (bf16 io); cont: add to the state given
based_status launch_state_generic_tc(const void* k, const void* v, float* kv, float* z, int BH, int L, int d_feat,
                                     int d_v, int cont, cudaStream_t stream);
// block_state_tc.cu: block states of the block-wise backward pass (d' = 16, bf16), transposed: st [BH x nblk][d_v][160]
// bf16 and sv [BH x nblk][160]: for every block of W tokens the sums over the blocks before it (rev = 0) or after it
// (rev = 1), one CTA per head; stats: (1 / D, b) per
// token for the query side (x = q, val = dout), null for the key side (x = k, val = v); part, zpart: null, or the
// blocks' own sums in fp32 instead (one CTA per head and block), for state_scan_kernel
based_status launch_block_states_tc(const void* x, const void* val, const void* stats, void* st, float* sv, float* part,
                                    float* zpart, int BH, int L, int W, int d_v, int rev, cudaStream_t stream);
// the state of a token block alone (no outputs): kv (+)= sum_j phi(k_j) v_j^T, z (+)= sum_j phi(k_j)
based_status launch_state_generic(const void* k, const void* v, float* kv, float* z, int BH, int L, int d_feat, int d_v,
                                  based_dtype io, int cont, cudaStream_t stream);
size_t prefill_tc_state_workspace_bytes(int BH, int L, int d_v);
based_status launch_prefill_tc_state(const void* k, const void* v, float* kv, float* z, int BH, int L, int d_v,
                                     int flags, void* workspace, cudaStream_t stream);
based_status launch_decode_generic(const void* q, const void* k, const void* v, float* kv, float* z, void* out,
                                   int BH, int d_feat, int d_v, based_dtype io, bool numerator_only,
                                   cudaStream_t stream);
// the same on tensor cores (bf16 io); ws: backward_tc_workspace_bytes
size_t backward_tc_workspace_bytes(int BH, int L, int d_v);
// block length of the block-wise path for this shape, 0 where the tile path runs (merged: forward output given, or
// the numerator-only form)
int backward_tc_block_tokens(int BH, int L, int d_feat, int d_v, int merged);
// out: the forward output (may be null): with it, statistics and dq run as one sweep
based_status launch_prefill_backward_tc(const void* q, const void* k, const void* v, const void* out, const void* g,
                                        void* dq, void* dk, void* dv, float* ws, int BH, int L, int d_feat, int d_v,
                                        int numerator_only, cudaStream_t stream);
// definition-form forward on tensor cores for d' in {8, 24, 32} (bf16 io, empty initial state)
based_status launch_quadratic_forward_tc(const void* q, const void* k, const void* v, void* out, int BH, int L,
                                         int d_feat, int d_v, int numerator_only, cudaStream_t stream);
// load the generation-step kernels into the current context
based_status preload_decode();
based_status preload_swa_decode();
based_status launch_swa_simt(const void* q, const void* k, const void* v, void* out, int BH, int L, int window,
                             float scale, based_dtype io, cudaStream_t stream);

}  // namespace based
