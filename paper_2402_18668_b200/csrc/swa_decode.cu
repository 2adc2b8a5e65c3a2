// swa_decode_step: one generation step of the sliding-window softmax mixer on a rolling cache
// of the last `window` keys and values (the PyTorch sliding-window listing and Algorithm 3 of
// App. B.2, here with the cache update included and for any position of the ring).
//
// One CTA of four warps per (b, h).  Thread 0 fetches the head's valid cache rows and the new q, k,
// v with five untiled bulk copies that complete on one mbarrier, so a head's whole
// 2 * window * 64 elements are in flight from the first instruction and up to 13 heads per SM
// stream at once.  The warps then work from shared memory: 8 lanes share a row (8 columns each),
// 4 rows per pass, passes dealt round-robin to the warps; scores are reduced with three shuffles
// and kept in registers; each warp forms the softmax numerator and denominator of its own rows
// relative to their maximum, and one block-wide barrier later the four partial results are
// rescaled and added.  The new k, v replace the row of slot pos % window on the fly and are
// stored to the cache.  The step reads the cache once: it is bound by HBM bandwidth and, at small
// batch, by launch latency.
#include "swa_decode.cuh"

namespace based {

using namespace swa_dec;

template <typename T, int NPW>
__global__ void __launch_bounds__(32 * kWarps)
swa_decode_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v, T* __restrict__ kc,
                  T* __restrict__ vc, T* __restrict__ out, int window, int pos_arg,
                  const int* pos_dev, int* pos_adv, float scale, unsigned int* __restrict__ error_word, int pos_group) {
    extern __shared__ __align__(128) unsigned char smem[];
    swa_decode_body<T, NPW, 1>(q, k, v, kc, vc, out, window, pos_arg, pos_dev, pos_adv, scale, error_word, blockIdx.x,
                               threadIdx.x, (int)gridDim.x, smem, pos_group);
}

template <typename T, int NPW>
static based_status launch_n(const void* q, const void* k, const void* v, void* kc, void* vc, void* out, int BH,
                             int window, int pos, const int* pos_dev, int* pos_adv, float scale, unsigned int* err,
                             cudaStream_t stream, int pos_group) {
    const size_t smem = swa_decode_smem_bytes<T>(window);
    if (smem > 48 * 1024) {
        if (cudaFuncSetAttribute(swa_decode_kernel<T, NPW>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem) != cudaSuccess)
            return BASED_ERR_CUDA;
    }
    swa_decode_kernel<T, NPW><<<BH, 32 * kWarps, smem, stream>>>(static_cast<const T*>(q), static_cast<const T*>(k),
                                                          static_cast<const T*>(v), static_cast<T*>(kc),
                                                          static_cast<T*>(vc), static_cast<T*>(out), window, pos,
                                                          pos_dev, pos_adv, scale, err, pos_group);
    note_launch();
    return check_launch("swa_decode_kernel");
}

template <typename T>
static based_status launch_t(const void* q, const void* k, const void* v, void* kc, void* vc, void* out, int BH,
                             int window, int pos, const int* pos_dev, int* pos_adv, float scale, unsigned int* err,
                             cudaStream_t stream, int pos_group) {
    if (window <= 64) return launch_n<T, 4>(q, k, v, kc, vc, out, BH, window, pos, pos_dev, pos_adv, scale, err, stream, pos_group);
    return launch_n<T, 8>(q, k, v, kc, vc, out, BH, window, pos, pos_dev, pos_adv, scale, err, stream, pos_group);
}

based_status preload_swa_decode() {
    cudaFuncAttributes attr;
    const bool ok = cudaFuncGetAttributes(&attr, swa_decode_kernel<float, 4>) == cudaSuccess &&
                    cudaFuncGetAttributes(&attr, swa_decode_kernel<float, 8>) == cudaSuccess &&
                    cudaFuncGetAttributes(&attr, swa_decode_kernel<__nv_bfloat16, 4>) == cudaSuccess &&
                    cudaFuncGetAttributes(&attr, swa_decode_kernel<__nv_bfloat16, 8>) == cudaSuccess;
    return ok ? BASED_OK : BASED_ERR_CUDA;
}

based_status launch_swa_decode(const void* q, const void* k, const void* v, void* kc, void* vc, void* out, int BH,
                               int window, int pos, const int* pos_dev, int* pos_adv, float scale, based_dtype io,
                               cudaStream_t stream, int pos_group) {
    unsigned int* err = nullptr;
    const based_status st = error_word_ptr(&err);
    if (st != BASED_OK) return st;
    if (io == BASED_F32)
        return launch_t<float>(q, k, v, kc, vc, out, BH, window, pos, pos_dev, pos_adv, scale, err, stream, pos_group);
    return launch_t<__nv_bfloat16>(q, k, v, kc, vc, out, BH, window, pos, pos_dev, pos_adv, scale, err, stream, pos_group);
}

}  // namespace based
