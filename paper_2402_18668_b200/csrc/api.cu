// C ABI of libbased: argument validation and dispatch.  See include/based.h for the
// contract of every entry point.
#include <atomic>
#include <mutex>
#include <cstdio>

#include "common.cuh"

namespace based {

__device__ unsigned int g_error_word = 0;

based_status error_word_ptr(unsigned int** ptr) {
    // the symbol has one instance per device: resolve it once per device, with that device current
    static std::atomic<unsigned int*> cache[64];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BASED_ERR_CUDA;
    unsigned int* p = cache[dev].load(std::memory_order_acquire);
    if (p == nullptr) {
        void* q = nullptr;
        if (cudaGetSymbolAddress(&q, g_error_word) != cudaSuccess) return BASED_ERR_CUDA;
        p = static_cast<unsigned int*>(q);
        cache[dev].store(p, std::memory_order_release);
    }
    *ptr = p;
    return BASED_OK;
}

std::mutex& setup_mutex() {
    static std::mutex mu;
    return mu;
}

static std::atomic<unsigned long long> g_launches{0};

void note_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

based_status check_launch(const char* what) {
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        std::fprintf(stderr, "libbased: launch of %s failed: %s\n", what, cudaGetErrorString(e));
        return BASED_ERR_CUDA;
    }
    return BASED_OK;
}

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
// value head dimensions: 64 (360M-scale heads), 128, and 112 (the 1.3B configuration's 1792 / 16)
static inline bool dv_ok(int d_v) { return d_v == 64 || d_v == 112 || d_v == 128; }
// feature dimensions of the paper's ablation other than 16: served by the fp32 definition-form kernels
static inline bool df_generic(int d_feat) { return d_feat == 8 || d_feat == 24 || d_feat == 32; }

}  // namespace based

using namespace based;

// Several kernels index heads by the y dimension of the grid (at most 65535).  Larger batches are cut into
// slabs of heads here: every tensor is [B*H, ...] with the heads outermost, so a slab is a contiguous piece,
// and the slabs run one after another on the caller's stream (sharing the caller's workspace, which is sized
// for the largest slab).
constexpr long long kHeadSlab = 65532;      // a multiple of 4: a slab's K-state (an odd number of floats per head) stays 16-byte aligned
static inline const void* off(const void* p, size_t bytes) { return p ? static_cast<const char*>(p) + bytes : nullptr; }
static inline void* off(void* p, size_t bytes) { return p ? static_cast<char*>(p) + bytes : nullptr; }
static inline float* off(float* p, size_t floats) { return p ? p + floats : nullptr; }
static inline size_t esize(based_dtype io) { return io == BASED_BF16 ? 2 : 4; }

extern "C" {

int based_version(void) { return 1; }

unsigned long long based_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* based_status_string(based_status s) {
    switch (s) {
        case BASED_OK: return "ok";
        case BASED_ERR_INVALID_ARG: return "invalid argument";
        case BASED_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case BASED_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case BASED_ERR_CUDA: return "CUDA error";
        case BASED_ERR_DEVICE_TIMEOUT: return "bounded device-side wait timed out";
        case BASED_ERR_WORKSPACE: return "workspace missing or too small";
    }
    return "unknown status";
}

size_t based_prefill_workspace_bytes(int B, int H, int L, int d_feat, int d_v, based_dtype io) {
    if (B <= 0 || H <= 0 || L <= 0 || d_feat != kDFeat || !dv_ok(d_v)) return 0;
    if (io != BASED_BF16) return 0;            // the fp32 path keeps its state in registers
    const long long BH = (long long)B * H;
    if (BH > kHeadSlab) {
        const size_t a = prefill_tc_workspace_bytes((int)kHeadSlab, L, d_v);
        const size_t b = BH % kHeadSlab ? prefill_tc_workspace_bytes((int)(BH % kHeadSlab), L, d_v) : 0;
        return a > b ? a : b;
    }
    return prefill_tc_workspace_bytes(B * H, L, d_v);
}

static based_status prefill_impl(const void* q, const void* k, const void* v, void* out, float* kv_state, float* z_state,
                                 int B, int H, int L, int d_feat, int d_v, based_dtype io, int flags, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream, bool fit) {
    if (!q || !k || !v || !out || B <= 0 || H <= 0 || L <= 0) return BASED_ERR_INVALID_ARG;
    if (io != BASED_F32 && io != BASED_BF16) return BASED_ERR_INVALID_ARG;
    if (flags & ~(BASED_STATE_CONTINUE | BASED_STATE_SYM | BASED_NUMERATOR_ONLY)) return BASED_ERR_INVALID_ARG;
    if ((kv_state == nullptr) != (z_state == nullptr)) return BASED_ERR_INVALID_ARG;
    if ((flags & BASED_STATE_CONTINUE) && !kv_state) return BASED_ERR_INVALID_ARG;
    if (out == q || out == k || out == v) return BASED_ERR_INVALID_ARG;
    if ((d_feat != kDFeat && !df_generic(d_feat)) || !dv_ok(d_v)) return BASED_ERR_UNSUPPORTED;
    if ((long long)B * H > 0x7fffffffLL) return BASED_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(kv_state) ||
        !aligned16(z_state) || !aligned16(workspace))
        return BASED_ERR_ALIGNMENT;
    if ((long long)B * H > kHeadSlab) {
        const size_t es = esize(io), rows = (flags & BASED_STATE_SYM) ? kDSym : 1 + d_feat + d_feat * d_feat;
        for (long long h0 = 0; h0 < (long long)B * H; h0 += kHeadSlab) {
            const int n = (int)((long long)B * H - h0 < kHeadSlab ? (long long)B * H - h0 : kHeadSlab);
            const based_status st = prefill_impl(
                off(q, (size_t)h0 * L * d_feat * es), off(k, (size_t)h0 * L * d_feat * es), off(v, (size_t)h0 * L * d_v * es),
                off(out, (size_t)h0 * L * d_v * es), off(kv_state, (size_t)h0 * rows * d_v), off(z_state, (size_t)h0 * rows),
                1, n, L, d_feat, d_v, io, flags, workspace, workspace_bytes, cuda_stream, fit);
            if (st != BASED_OK) return st;
        }
        return BASED_OK;
    }
    if (d_feat != kDFeat) {
        if (flags & BASED_STATE_SYM) return BASED_ERR_UNSUPPORTED;
        // bf16 io from the empty state: outputs on the tensor cores (definition form), the state by the fp32 kernel
        bool outputs_done = false;
        if (io == BASED_BF16 && !(flags & BASED_STATE_CONTINUE)) {
            const based_status st =
                launch_quadratic_forward_tc(q, k, v, out, B * H, L, d_feat, d_v, (flags & BASED_NUMERATOR_ONLY) ? 1 : 0,
                                            static_cast<cudaStream_t>(cuda_stream));
            if (st != BASED_OK) return st;
            outputs_done = true;
        }
        return launch_prefill_generic(q, k, v, out, kv_state, z_state, B * H, L, d_feat, d_v, io, flags, outputs_done,
                                      static_cast<cudaStream_t>(cuda_stream));
    }
    const size_t need = based_prefill_workspace_bytes(B, H, L, d_feat, d_v, io);
    if (!fit && need > 0 && (!workspace || workspace_bytes < need)) return BASED_ERR_WORKSPACE;
    if (io == BASED_BF16)
        return launch_prefill_tc(q, k, v, out, kv_state, z_state, B * H, L, d_v, flags, workspace,
                                 static_cast<cudaStream_t>(cuda_stream), fit ? workspace_bytes : ~(size_t)0);
    return launch_prefill_simt(q, k, v, out, kv_state, z_state, B * H, L, d_v, io, flags,
                               static_cast<cudaStream_t>(cuda_stream));
}

based_status based_prefill(const void* q, const void* k, const void* v, void* out, float* kv_state, float* z_state,
                           int B, int H, int L, int d_feat, int d_v, based_dtype io, int flags, void* workspace,
                           size_t workspace_bytes, void* cuda_stream) {
    return prefill_impl(q, k, v, out, kv_state, z_state, B, H, L, d_feat, d_v, io, flags, workspace, workspace_bytes,
                        cuda_stream, false);
}

size_t based_prefill_state_workspace_bytes(int B, int H, int L, int d_feat, int d_v, based_dtype io) {
    if (B <= 0 || H <= 0 || L <= 0 || d_feat != kDFeat || !dv_ok(d_v) || io != BASED_BF16) return 0;
    if ((long long)B * H > kHeadSlab) return prefill_tc_state_workspace_bytes((int)kHeadSlab, L, d_v);   // heads x one partial state: the largest slab's
    return prefill_tc_state_workspace_bytes(B * H, L, d_v);
}

based_status based_prefill_state(const void* k, const void* v, float* kv_state, float* z_state, int B, int H, int L,
                                 int d_feat, int d_v, based_dtype io, int flags, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream) {
    if (!k || !v || !kv_state || !z_state || B <= 0 || H <= 0 || L <= 0) return BASED_ERR_INVALID_ARG;
    if (io != BASED_F32 && io != BASED_BF16) return BASED_ERR_INVALID_ARG;
    if (flags & ~(BASED_STATE_CONTINUE | BASED_STATE_SYM)) return BASED_ERR_INVALID_ARG;
    if ((d_feat != kDFeat && !df_generic(d_feat)) || !dv_ok(d_v)) return BASED_ERR_UNSUPPORTED;
    if ((long long)B * H > 0x7fffffffLL) return BASED_ERR_UNSUPPORTED;
    const bool tc16 = d_feat == kDFeat && io == BASED_BF16;
    if ((flags & BASED_STATE_SYM) && !tc16) return BASED_ERR_UNSUPPORTED;      // symmetric rows: d' = 16, bf16 io
    if (!aligned16(k) || !aligned16(v) || !aligned16(kv_state) || !aligned16(z_state) || !aligned16(workspace))
        return BASED_ERR_ALIGNMENT;
    if ((long long)B * H > kHeadSlab) {
        const size_t es = esize(io), rows = (flags & BASED_STATE_SYM) ? kDSym : 1 + d_feat + d_feat * d_feat;
        for (long long h0 = 0; h0 < (long long)B * H; h0 += kHeadSlab) {
            const int n = (int)((long long)B * H - h0 < kHeadSlab ? (long long)B * H - h0 : kHeadSlab);
            const based_status st = based_prefill_state(
                off(k, (size_t)h0 * L * d_feat * es), off(v, (size_t)h0 * L * d_v * es), off(kv_state, (size_t)h0 * rows * d_v),
                off(z_state, (size_t)h0 * rows), 1, n, L, d_feat, d_v, io, flags, workspace, workspace_bytes, cuda_stream);
            if (st != BASED_OK) return st;
        }
        return BASED_OK;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (tc16) {
        if (!workspace || workspace_bytes < based_prefill_state_workspace_bytes(B, H, L, d_feat, d_v, io))
            return BASED_ERR_WORKSPACE;
        return launch_prefill_tc_state(k, v, kv_state, z_state, B * H, L, d_v, flags, workspace, stream);
    }
    return launch_state_generic(k, v, kv_state, z_state, B * H, L, d_feat, d_v, io,
                                (flags & BASED_STATE_CONTINUE) ? 1 : 0, stream);
}

based_status based_decode_step(const void* q, const void* k, const void* v, float* kv_state, float* z_state,
                               void* out, int B, int H, int d_feat, int d_v, based_dtype io, void* cuda_stream) {
    if (!q || !k || !v || !out || !kv_state || !z_state || B <= 0 || H <= 0) return BASED_ERR_INVALID_ARG;
    if (io != BASED_F32 && io != BASED_BF16) return BASED_ERR_INVALID_ARG;
    if ((d_feat != kDFeat && !df_generic(d_feat)) || !dv_ok(d_v)) return BASED_ERR_UNSUPPORTED;
    if ((long long)B * H > 0x7fffffffLL) return BASED_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(kv_state) ||
        !aligned16(z_state))
        return BASED_ERR_ALIGNMENT;
    if (d_feat != kDFeat)
        return launch_decode_generic(q, k, v, kv_state, z_state, out, B * H, d_feat, d_v, io, false,
                                     static_cast<cudaStream_t>(cuda_stream));
    return launch_decode(q, k, v, kv_state, z_state, out, B * H, d_v, io, false, false,
                         static_cast<cudaStream_t>(cuda_stream));
}

based_status based_decode_step_flags(const void* q, const void* k, const void* v, float* kv_state, float* z_state,
                                     void* out, int B, int H, int d_feat, int d_v, based_dtype io, int flags,
                                     void* cuda_stream) {
    if (!q || !k || !v || !out || !kv_state || !z_state || B <= 0 || H <= 0) return BASED_ERR_INVALID_ARG;
    if (io != BASED_F32 && io != BASED_BF16) return BASED_ERR_INVALID_ARG;
    if (flags & ~(BASED_STATE_SYM | BASED_NUMERATOR_ONLY)) return BASED_ERR_INVALID_ARG;
    if ((d_feat != kDFeat && !df_generic(d_feat)) || !dv_ok(d_v)) return BASED_ERR_UNSUPPORTED;
    if ((long long)B * H > 0x7fffffffLL) return BASED_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(kv_state) ||
        !aligned16(z_state))
        return BASED_ERR_ALIGNMENT;
    if (d_feat != kDFeat) {
        if (flags & BASED_STATE_SYM) return BASED_ERR_UNSUPPORTED;
        return launch_decode_generic(q, k, v, kv_state, z_state, out, B * H, d_feat, d_v, io,
                                     (flags & BASED_NUMERATOR_ONLY) != 0, static_cast<cudaStream_t>(cuda_stream));
    }
    return launch_decode(q, k, v, kv_state, z_state, out, B * H, d_v, io, (flags & BASED_STATE_SYM) != 0,
                         (flags & BASED_NUMERATOR_ONLY) != 0, static_cast<cudaStream_t>(cuda_stream));
}

based_status based_decode_step_sym(const void* q, const void* k, const void* v, float* kv_sym, float* z_sym,
                                   void* out, int B, int H, int d_feat, int d_v, based_dtype io,
                                   void* cuda_stream) {
    if (!q || !k || !v || !out || !kv_sym || !z_sym || B <= 0 || H <= 0) return BASED_ERR_INVALID_ARG;
    if (io != BASED_F32 && io != BASED_BF16) return BASED_ERR_INVALID_ARG;
    if (d_feat != kDFeat || !dv_ok(d_v)) return BASED_ERR_UNSUPPORTED;
    if ((long long)B * H > 0x7fffffffLL) return BASED_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(kv_sym) ||
        !aligned16(z_sym))
        return BASED_ERR_ALIGNMENT;
    return launch_decode(q, k, v, kv_sym, z_sym, out, B * H, d_v, io, true, false,
                         static_cast<cudaStream_t>(cuda_stream));
}

static based_status state_convert(const float* kv_in, const float* z_in, float* kv_out, float* z_out, int B, int H,
                                  int d_feat, int d_v, bool to_sym, void* cuda_stream) {
    if (!kv_in || !z_in || !kv_out || !z_out || B <= 0 || H <= 0) return BASED_ERR_INVALID_ARG;
    if (kv_in == kv_out || z_in == z_out) return BASED_ERR_INVALID_ARG;
    if (d_feat != kDFeat || !dv_ok(d_v)) return BASED_ERR_UNSUPPORTED;
    if ((long long)B * H > 0x7fffffffLL) return BASED_ERR_UNSUPPORTED;
    if (!aligned16(kv_in) || !aligned16(z_in) || !aligned16(kv_out) || !aligned16(z_out)) return BASED_ERR_ALIGNMENT;
    return launch_state_convert(kv_in, z_in, kv_out, z_out, B * H, d_v, to_sym,
                                static_cast<cudaStream_t>(cuda_stream));
}

based_status based_state_to_sym(const float* kv_state, const float* z_state, float* kv_sym, float* z_sym, int B,
                                int H, int d_feat, int d_v, void* cuda_stream) {
    return state_convert(kv_state, z_state, kv_sym, z_sym, B, H, d_feat, d_v, true, cuda_stream);
}

based_status based_state_from_sym(const float* kv_sym, const float* z_sym, float* kv_state, float* z_state, int B,
                                  int H, int d_feat, int d_v, void* cuda_stream) {
    return state_convert(kv_sym, z_sym, kv_state, z_state, B, H, d_feat, d_v, false, cuda_stream);
}

based_status swa_forward(const void* q, const void* k, const void* v, void* out, int B, int H, int L, int d,
                         int window, float softmax_scale, based_dtype io, void* cuda_stream) {
    if (!q || !k || !v || !out || B <= 0 || H <= 0 || L <= 0 || window <= 0) return BASED_ERR_INVALID_ARG;
    if (io != BASED_F32 && io != BASED_BF16) return BASED_ERR_INVALID_ARG;
    if (out == q || out == k || out == v) return BASED_ERR_INVALID_ARG;
    if (d != 64 || window > 128) return BASED_ERR_UNSUPPORTED;
    if ((long long)B * H > 0x7fffffffLL) return BASED_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return BASED_ERR_ALIGNMENT;
    if ((long long)B * H > kHeadSlab) {
        const size_t hb = (size_t)L * d * esize(io);
        for (long long h0 = 0; h0 < (long long)B * H; h0 += kHeadSlab) {
            const int n = (int)((long long)B * H - h0 < kHeadSlab ? (long long)B * H - h0 : kHeadSlab);
            const based_status st = swa_forward(off(q, h0 * hb), off(k, h0 * hb), off(v, h0 * hb), off(out, h0 * hb), 1, n, L,
                                                d, window, softmax_scale, io, cuda_stream);
            if (st != BASED_OK) return st;
        }
        return BASED_OK;
    }
    const float scale = softmax_scale > 0.f ? softmax_scale : 0.125f;   // 1/sqrt(64)
    if (io == BASED_BF16 && swa_tc_supported(window))
        return launch_swa_tc(q, k, v, out, B * H, L, window, scale, static_cast<cudaStream_t>(cuda_stream));
    return launch_swa_simt(q, k, v, out, B * H, L, window, scale, io, static_cast<cudaStream_t>(cuda_stream));
}

based_status swa_decode_step(const void* q, const void* k, const void* v, void* k_cache, void* v_cache, void* out,
                             int B, int H, int d, int window, int pos, float softmax_scale, based_dtype io,
                             void* cuda_stream) {
    if (!q || !k || !v || !k_cache || !v_cache || !out || B <= 0 || H <= 0 || window <= 0 || pos < 0)
        return BASED_ERR_INVALID_ARG;
    if (io != BASED_F32 && io != BASED_BF16) return BASED_ERR_INVALID_ARG;
    if (d != 64 || window > 128) return BASED_ERR_UNSUPPORTED;
    if ((long long)B * H > 0x7fffffffLL) return BASED_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(k_cache) || !aligned16(v_cache) ||
        !aligned16(out))
        return BASED_ERR_ALIGNMENT;
    const float scale = softmax_scale > 0.f ? softmax_scale : 0.125f;   // 1/sqrt(64)
    return launch_swa_decode(q, k, v, k_cache, v_cache, out, B * H, window, pos, nullptr, nullptr, scale, io,
                             static_cast<cudaStream_t>(cuda_stream));
}

based_status swa_decode_step_at(const void* q, const void* k, const void* v, void* k_cache, void* v_cache,
                                void* out, int B, int H, int d, int window, const int* pos_device,
                                float softmax_scale, based_dtype io, void* cuda_stream) {
    if (!q || !k || !v || !k_cache || !v_cache || !out || !pos_device || B <= 0 || H <= 0 || window <= 0)
        return BASED_ERR_INVALID_ARG;
    if (io != BASED_F32 && io != BASED_BF16) return BASED_ERR_INVALID_ARG;
    if (d != 64 || window > 128) return BASED_ERR_UNSUPPORTED;
    if ((long long)B * H > 0x7fffffffLL) return BASED_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(k_cache) || !aligned16(v_cache) ||
        !aligned16(out) || (reinterpret_cast<uintptr_t>(pos_device) & 3u))
        return BASED_ERR_ALIGNMENT;
    const float scale = softmax_scale > 0.f ? softmax_scale : 0.125f;   // 1/sqrt(64)
    return launch_swa_decode(q, k, v, k_cache, v_cache, out, B * H, window, 0, pos_device, nullptr, scale, io,
                             static_cast<cudaStream_t>(cuda_stream));
}

based_status swa_decode_step_ragged(const void* q, const void* k, const void* v, void* k_cache, void* v_cache,
                                    void* out, int B, int H, int d, int window, const int* pos_per_sequence,
                                    float softmax_scale, based_dtype io, void* cuda_stream) {
    if (!q || !k || !v || !k_cache || !v_cache || !out || !pos_per_sequence || B <= 0 || H <= 0 || window <= 0)
        return BASED_ERR_INVALID_ARG;
    if (io != BASED_F32 && io != BASED_BF16) return BASED_ERR_INVALID_ARG;
    if (d != 64 || window > 128) return BASED_ERR_UNSUPPORTED;
    if ((long long)B * H > 0x7fffffffLL) return BASED_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(k_cache) || !aligned16(v_cache) ||
        !aligned16(out) || (reinterpret_cast<uintptr_t>(pos_per_sequence) & 3u))
        return BASED_ERR_ALIGNMENT;
    const float scale = softmax_scale > 0.f ? softmax_scale : 0.125f;   // 1/sqrt(64)
    return launch_swa_decode(q, k, v, k_cache, v_cache, out, B * H, window, 0, pos_per_sequence, nullptr, scale, io,
                             static_cast<cudaStream_t>(cuda_stream), H);
}

based_status swa_decode_step_advance(const void* q, const void* k, const void* v, void* k_cache, void* v_cache,
                                     void* out, int B, int H, int d, int window, int* pos_state,
                                     float softmax_scale, based_dtype io, void* cuda_stream) {
    if (!q || !k || !v || !k_cache || !v_cache || !out || !pos_state || B <= 0 || H <= 0 || window <= 0)
        return BASED_ERR_INVALID_ARG;
    if (io != BASED_F32 && io != BASED_BF16) return BASED_ERR_INVALID_ARG;
    if (d != 64 || window > 128) return BASED_ERR_UNSUPPORTED;
    if ((long long)B * H > 0x7fffffffLL) return BASED_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(k_cache) || !aligned16(v_cache) ||
        !aligned16(out) || (reinterpret_cast<uintptr_t>(pos_state) & 7u))
        return BASED_ERR_ALIGNMENT;
    const float scale = softmax_scale > 0.f ? softmax_scale : 0.125f;   // 1/sqrt(64)
    return launch_swa_decode(q, k, v, k_cache, v_cache, out, B * H, window, 0, pos_state, pos_state, scale, io,
                             static_cast<cudaStream_t>(cuda_stream));
}

based_status based_generation_step(const void* q, const void* k, const void* v, float* kv_state, float* z_state,
                                   void* out, const void* qw, const void* kw, const void* vw, void* k_cache,
                                   void* v_cache, void* out_w, int B, int H, int d_feat, int d_v, int H_w, int d_w,
                                   int window, int* pos_state, float softmax_scale, based_dtype io, int flags,
                                   void* cuda_stream) {
    if (!q || !k || !v || !kv_state || !z_state || !out || !qw || !kw || !vw || !k_cache || !v_cache || !out_w ||
        !pos_state || B <= 0 || H <= 0 || H_w <= 0 || window <= 0)
        return BASED_ERR_INVALID_ARG;
    if (io != BASED_F32 && io != BASED_BF16) return BASED_ERR_INVALID_ARG;
    if (flags & ~(BASED_STATE_SYM | BASED_NUMERATOR_ONLY)) return BASED_ERR_INVALID_ARG;
    if (d_feat != kDFeat || !dv_ok(d_v) || d_w != 64 || window > 128) return BASED_ERR_UNSUPPORTED;
    if ((long long)B * H + ((long long)B * H_w + 1) / 2 > 0x7fffffffLL) return BASED_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(kv_state) || !aligned16(z_state) ||
        !aligned16(out) || !aligned16(qw) || !aligned16(kw) || !aligned16(vw) || !aligned16(k_cache) ||
        !aligned16(v_cache) || !aligned16(out_w) || (reinterpret_cast<uintptr_t>(pos_state) & 7u))
        return BASED_ERR_ALIGNMENT;
    const float scale = softmax_scale > 0.f ? softmax_scale : 0.125f;   // 1/sqrt(64)
    return launch_generation_step(q, k, v, kv_state, z_state, out, B * H, d_v, (flags & BASED_STATE_SYM) != 0,
                                  (flags & BASED_NUMERATOR_ONLY) != 0, qw, kw, vw, k_cache, v_cache, out_w, B * H_w,
                                  window, pos_state, scale, io, static_cast<cudaStream_t>(cuda_stream));
}

static based_status baseconv_check(const void* a, const void* g, const float* h, const float* b2, const void* out,
                                   int B, int N, int C, int width, based_dtype io) {
    if (!a || !g || !h || !b2 || !out || B <= 0 || N <= 0 || C <= 0 || width <= 0) return BASED_ERR_INVALID_ARG;
    if (io != BASED_F32 && io != BASED_BF16) return BASED_ERR_INVALID_ARG;
    if (out == g) return BASED_ERR_INVALID_ARG;
    if (width > 4 || C % 8 != 0 || B > 65535 || (N + 63) / 64 > 65535) return BASED_ERR_UNSUPPORTED;
    if (!aligned16(a) || !aligned16(g) || !aligned16(h) || !aligned16(b2) || !aligned16(out)) return BASED_ERR_ALIGNMENT;
    return BASED_OK;
}

based_status baseconv_gate_forward(const void* a, const void* g, const float* h, const float* b2, void* out, int B,
                                   int N, int C, int width, based_dtype io, void* cuda_stream) {
    const based_status st = baseconv_check(a, g, h, b2, out, B, N, C, width, io);
    if (st != BASED_OK) return st;
    return launch_baseconv(a, g, h, b2, nullptr, out, B, N, C, width, false, io,
                           static_cast<cudaStream_t>(cuda_stream));
}

based_status baseconv_gate_step(const void* a, const void* g, const float* h, const float* b2, void* conv_state,
                                void* out, int B, int C, int width, based_dtype io, void* cuda_stream) {
    const based_status st = baseconv_check(a, g, h, b2, out, B, 1, C, width, io);
    if (st != BASED_OK) return st;
    if (width > 1 && !conv_state) return BASED_ERR_INVALID_ARG;
    if (!aligned16(conv_state)) return BASED_ERR_ALIGNMENT;
    return launch_baseconv(a, g, h, b2, conv_state, out, B, 1, C, width, true, io,
                           static_cast<cudaStream_t>(cuda_stream));
}

size_t based_prefill_backward_workspace_bytes(int B, int H, int L, int d_v, based_dtype io) {
    if (B <= 0 || H <= 0 || L <= 0 || !dv_ok(d_v)) return 0;
    const int heads = (long long)B * H > kHeadSlab ? (int)kHeadSlab : B * H;       // the largest slab of heads
    if (io == BASED_BF16) return backward_tc_workspace_bytes(heads, L, d_v);
    return (size_t)heads * L * 2 * sizeof(float);
}

int based_prefill_backward_block_tokens(int B, int H, int L, int d_feat, int d_v, based_dtype io, int flags,
                                        int with_out) {
    if (B <= 0 || H <= 0 || L <= 0 || !dv_ok(d_v) || io != BASED_BF16) return 0;
    return backward_tc_block_tokens(B * H, L, d_feat, d_v, (with_out || (flags & BASED_NUMERATOR_ONLY)) ? 1 : 0);
}

static based_status prefill_backward(const void* q, const void* k, const void* v, const void* out, const void* dout,
                                     void* dq, void* dk, void* dv, int B, int H, int L, int d_feat, int d_v,
                                     based_dtype io, int flags, void* workspace, size_t workspace_bytes,
                                     void* cuda_stream) {
    if (!q || !k || !v || !dout || !dq || !dk || !dv || B <= 0 || H <= 0 || L <= 0) return BASED_ERR_INVALID_ARG;
    if (io != BASED_F32 && io != BASED_BF16) return BASED_ERR_INVALID_ARG;
    if (flags & ~BASED_NUMERATOR_ONLY) return BASED_ERR_INVALID_ARG;
    if (dq == q || dq == k || dk == q || dk == k || dv == v || dv == dout) return BASED_ERR_INVALID_ARG;
    // the other feature dimensions: bf16 io only (the tensor-core kernels take d' as a parameter)
    if (!(d_feat == kDFeat || (df_generic(d_feat) && io == BASED_BF16)) || !dv_ok(d_v)) return BASED_ERR_UNSUPPORTED;
    if ((long long)B * H > 0x7fffffffLL) return BASED_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(dout) || !aligned16(dq) || !aligned16(dk) ||
        !aligned16(dv) || !aligned16(workspace) || !aligned16(out))
        return BASED_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < based_prefill_backward_workspace_bytes(B, H, L, d_v, io))
        return BASED_ERR_WORKSPACE;
    if ((long long)B * H > kHeadSlab) {
        const size_t qb = (size_t)L * d_feat * esize(io), vb = (size_t)L * d_v * esize(io);
        for (long long h0 = 0; h0 < (long long)B * H; h0 += kHeadSlab) {
            const int n = (int)((long long)B * H - h0 < kHeadSlab ? (long long)B * H - h0 : kHeadSlab);
            const based_status st = prefill_backward(off(q, h0 * qb), off(k, h0 * qb), off(v, h0 * vb), off(out, h0 * vb),
                                                     off(dout, h0 * vb), off(dq, h0 * qb), off(dk, h0 * qb), off(dv, h0 * vb), 1,
                                                     n, L, d_feat, d_v, io, flags, workspace, workspace_bytes, cuda_stream);
            if (st != BASED_OK) return st;
        }
        return BASED_OK;
    }
    if (io == BASED_BF16)
        return launch_prefill_backward_tc(q, k, v, out, dout, dq, dk, dv, static_cast<float*>(workspace), B * H, L,
                                          d_feat, d_v, (flags & BASED_NUMERATOR_ONLY) ? 1 : 0,
                                          static_cast<cudaStream_t>(cuda_stream));
    return launch_prefill_backward(q, k, v, dout, dq, dk, dv, static_cast<float*>(workspace), B * H, L, d_v, io,
                                   (flags & BASED_NUMERATOR_ONLY) ? 1 : 0, static_cast<cudaStream_t>(cuda_stream));
}

based_status based_prefill_backward(const void* q, const void* k, const void* v, const void* dout, void* dq,
                                    void* dk, void* dv, int B, int H, int L, int d_feat, int d_v, based_dtype io,
                                    int flags, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return prefill_backward(q, k, v, nullptr, dout, dq, dk, dv, B, H, L, d_feat, d_v, io, flags, workspace,
                            workspace_bytes, cuda_stream);
}

based_status based_prefill_backward_with_out(const void* q, const void* k, const void* v, const void* out,
                                             const void* dout, void* dq, void* dk, void* dv, int B, int H, int L,
                                             int d_feat, int d_v, based_dtype io, int flags, void* workspace,
                                             size_t workspace_bytes, void* cuda_stream) {
    if (!out || out == dq || out == dk || out == dv) return BASED_ERR_INVALID_ARG;
    return prefill_backward(q, k, v, out, dout, dq, dk, dv, B, H, L, d_feat, d_v, io, flags, workspace,
                            workspace_bytes, cuda_stream);
}

based_status based_preload_decode(void) {
    unsigned int* err = nullptr;
    based_status st = error_word_ptr(&err);
    if (st == BASED_OK) st = preload_decode();
    if (st == BASED_OK) st = preload_swa_decode();
    if (st == BASED_OK) st = preload_generation_step();
    return st;
}

based_status based_poll_error(void* cuda_stream) {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return BASED_ERR_CUDA;
    unsigned int word = 0;
    if (cudaMemcpyFromSymbol(&word, g_error_word, sizeof(word)) != cudaSuccess) return BASED_ERR_CUDA;
    if (word != 0) {
        const unsigned int zero = 0;
        if (cudaMemcpyToSymbol(g_error_word, &zero, sizeof(zero)) != cudaSuccess) return BASED_ERR_CUDA;
        return BASED_ERR_DEVICE_TIMEOUT;
    }
    return BASED_OK;
}

}  // extern "C"

namespace based {
based_status prefill_fit_workspace(const void* q, const void* k, const void* v, void* out, float* kv_state, float* z_state,
                                   int B, int H, int L, int d_feat, int d_v, based_dtype io, int flags, void* workspace,
                                   size_t workspace_bytes, void* cuda_stream) {
    return ::prefill_impl(q, k, v, out, kv_state, z_state, B, H, L, d_feat, d_v, io, flags, workspace, workspace_bytes,
                          cuda_stream, true);
}
}  // namespace based
