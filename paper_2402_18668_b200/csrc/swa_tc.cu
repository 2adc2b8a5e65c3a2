// swa_forward, bf16 tensor-core path (tcgen05 + TMEM + TMA): exact causal softmax
// attention in a sliding window (Eq. (1) of Sec. 2 with the key set {i-w+1..i} of
// Sec. 4.2), head dimension 64, window <= 128.
//
// Persistent CTAs (one per SM) walk tiles of 128 consecutive queries of one head.  The 192
// keys a tile can see (64 before its first query, then its own 128) are loaded once; per tile
//   S[128,192] = Q K^T          4 MMAs (K = 64), fp32 in TMEM
//   softmax    one thread per query row reads the 96 columns its warp's rows can touch,
//              masks to its own window, exp2 with the scale folded in, writes P (bf16) back
//              into TMEM over the scores
//   O[128,64]  = P V            12 MMAs with P read from TMEM
//   out        O / rowsum -> bf16 -> swizzled shared tile -> TMA store.
// The kernel is bound by HBM (512 B per token and head against ~50 k flop): a 3-stage TMA
// ring prefetches tiles, and two softmax groups with one TMEM buffer each alternate tiles so
// that loads, MMAs, softmax and stores of neighbouring tiles overlap.
//
// Windows of 65..128 keys run the same kernel with 128 keys before the tile (PAD = 128): 256 keys
// per tile, S[128,256] filling the tile's 256 tensor-memory columns, and a softmax in two passes
// over the 160 columns a warp's rows can touch (maximum first, then exponentials and the packed
// weights, 32 columns at a time, written over columns that have been read already).  Each CTA
// walks a contiguous run of tiles, so the 128 rows of K and V before a tile are the ones the tile
// before it loaded: a tile loads only its own rows (48 KB with Q) into one of four slots, and the
// MMAs address two slots (two N = 128 score products per K step, the P V steps over two V blocks).
#include <cuda_bf16.h>

#include "common.cuh"
#include "sm100.cuh"

namespace based {

using namespace sm100;

namespace {

constexpr int kQT = 128;                 // queries per tile
constexpr int kHD = 64;
constexpr int kThreads = 320;            // 2 softmax groups of 4 warps, TMA producer warp, MMA warp
constexpr int kWarpTma = 8, kWarpMma = 9;
constexpr uint32_t kQBytes = kQT * kHD * 2;      // 16 KB
// PAD: keys loaded before the tile's first query (>= window - 1): 64 or 128
template <int PAD> struct SwaCfg {
    static constexpr int kPad = PAD;
    static constexpr int kKeys = kQT + PAD;                        // 192 / 256 keys under a tile's scores
    // PAD 64: a stage holds a tile's Q and its 192 rows of K and of V.  PAD 128: a slot holds a tile's Q and its
    // own 128 rows of K and of V; the 128 rows before them are the previous tile's, still in the slot before.
    static constexpr int kStages = PAD == 64 ? 3 : 4;
    static constexpr uint32_t kKVBytes = (PAD == 64 ? kKeys : kQT) * kHD * 2;   // 24 / 16 KB
    static constexpr uint32_t kStageBytes = kQBytes + 2 * kKVBytes;   // 64 / 48 KB
    static constexpr uint32_t offOut = kStages * kStageBytes;      // two 16 KB output staging tiles (one per group)
    static constexpr uint32_t offBars = offOut + 2 * kQBytes;
    static constexpr uint32_t kSmemBytes = offBars + 256 + 1024;
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};
constexpr uint32_t kBufCols = 256;               // TMEM columns per tile in flight
constexpr uint32_t colS = 0, colO = 128;         // P overwrites the first half of S's columns; O uses dead S columns

enum SwaBar { bFull = 0, bEmpty = 4, bS = 8, bP = 10, bO = 12, bOfree = 14, bCount = 16 };

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ void group_sync(int id) {
    asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory");
}
__device__ __forceinline__ bool group_all(int id, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.and.pred q, %2, 128, p;\n\t"
        "selp.b32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred), "r"(id)
        : "memory");
    return r != 0;
}

struct SwaParams {
    unsigned int* err;
    int L;
    int window;
    int tiles_per_head;
    int total_tiles;
    float scale_log2e;      // softmax scale * log2(e)
};

}  // namespace

// Persistent kernel: CTA j handles tiles j, j + gridDim.x, ...  Tile n of a CTA uses shared
// memory stage n % 3 and TMEM buffer n % 2; softmax group n % 2 owns it.
template <int PAD>
__global__ void __launch_bounds__(kThreads, 1)
    swa_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                  const SwaParams p) {
    using C = SwaCfg<PAD>;
    constexpr int kPad = C::kPad, kKeys = C::kKeys, kStages = C::kStages;
    constexpr uint32_t kKVBytes = C::kKVBytes, kStageBytes = C::kStageBytes, offOut = C::offOut, offBars = C::offBars;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + offBars);
    uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(bars + bCount);
    volatile uint32_t* abort_flag = tmem_base_s + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // PAD 64: CTA j takes tiles j, j + gridDim.x, ...; PAD 128: a contiguous run of tiles, so that a tile's
    // first 128 keys are the rows the tile before it loaded
    const int run_first = (int)((long long)p.total_tiles * blockIdx.x / gridDim.x);
    const int run_last = (int)((long long)p.total_tiles * (blockIdx.x + 1) / gridDim.x);
    const int ntiles = PAD == 64 ? (p.total_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x
                                 : run_last - run_first;
    auto tile_of = [&](int n) -> int { return PAD == 64 ? (int)blockIdx.x + n * (int)gridDim.x : run_first + n; };

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&bars[bFull + s], 1); mbar_init(&bars[bEmpty + s], 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bars[bS + b], 1); mbar_init(&bars[bP + b], 128);
            mbar_init(&bars[bO + b], 1); mbar_init(&bars[bOfree + b], 128);
        }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v); prefetch_tensormap(&tm_o);
    }
    if (warp == kWarpMma) { tmem_alloc(tmem_base_s, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = *tmem_base_s;
    bool ok = true;

    if (warp == kWarpTma) {
        if (lane == 0) {
            if constexpr (PAD == 64) {
                for (int n = 0; n < ntiles && ok; ++n) {
                    const int s = n % kStages;
                    ok = mbar_wait(&bars[bEmpty + s], ((n / kStages) & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    const int tile = tile_of(n);
                    const int head = tile / p.tiles_per_head, i0 = (tile % p.tiles_per_head) * kQT;
                    uint8_t* st = smem + s * kStageBytes;
                    // Q tile, and K, V rows i0-PAD .. i0+127 (rows before the sequence start read as zero)
                    mbar_arrive_expect_tx(&bars[bFull + s], kStageBytes);
                    tma_load_3d(st, &tm_q, &bars[bFull + s], 0, i0, head);
                    tma_load_3d(st + kQBytes, &tm_k, &bars[bFull + s], 0, i0 - kPad, head);
                    tma_load_3d(st + kQBytes + kKVBytes, &tm_v, &bars[bFull + s], 0, i0 - kPad, head);
                }
            } else {
                // load m = 0: the 128 rows of K and V before the run's first tile (zeros at a head's start);
                // load m >= 1: Q, K, V rows of tile m - 1.  Slot m % 4; a slot is free once the tile that
                // used it as "rows before" has finished its P V products.
                for (int m = 0; m <= ntiles && ok && ntiles > 0; ++m) {
                    const int s = m % kStages;
                    ok = mbar_wait(&bars[bEmpty + s], ((m / kStages) & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    const int tile = tile_of(m == 0 ? 0 : m - 1);
                    const int head = tile / p.tiles_per_head;
                    const int i0 = (tile % p.tiles_per_head) * kQT - (m == 0 ? kQT : 0);
                    uint8_t* st = smem + s * kStageBytes;
                    mbar_arrive_expect_tx(&bars[bFull + s], m == 0 ? 2 * kKVBytes : kStageBytes);
                    if (m > 0) tma_load_3d(st, &tm_q, &bars[bFull + s], 0, i0, head);
                    tma_load_3d(st + kQBytes, &tm_k, &bars[bFull + s], 0, i0, head);
                    tma_load_3d(st + kQBytes + kKVBytes, &tm_v, &bars[bFull + s], 0, i0, head);
                }
            }
        }
    } else if (warp == kWarpMma) {
        {
            // the whole warp runs this block and one elected lane issues (see mma_ss_w)
            const uint32_t lead = elect_one();
            constexpr uint64_t dK = make_smem_desc_base(16, 1024, kSwizzle128B);   // K-major rows / MN-major block
            constexpr uint32_t iS = make_idesc_bf16(kQT, kKeys, 0, 0);
            constexpr uint32_t iO = make_idesc_bf16(kQT, kHD, 0, 1);
            if constexpr (PAD == 64) {
                auto issue_pv = [&](int n) {
                    const uint32_t tbuf = tb + (n & 1) * kBufCols;
                    const uint32_t lV = desc_lo(dK) + (smem_u32(smem + (n % kStages) * kStageBytes + kQBytes + kKVBytes) >> 4);
                    mma_ts_w<false>(lead, tbuf + colO, tbuf + colS, lV, desc_hi(dK), iO);
#pragma unroll
                    for (int k = 1; k < kKeys / 16; ++k)
                        mma_ts_w<true>(lead, tbuf + colO, tbuf + colS + k * 8, lV + k * (2048 >> 4), desc_hi(dK), iO);
                    mma_commit_w(lead, &bars[bO + (n & 1)]);
                    mma_commit_w(lead, &bars[bEmpty + n % kStages]);     // K, V (and Q) of this stage are dead
                };
                for (int n = 0; n < ntiles && ok; ++n) {
                    const int s = n % kStages, b = n & 1;
                    ok = mbar_wait(&bars[bFull + s], (n / kStages) & 1, abort_flag);
                    // the buffer's previous tile (n - 2) must have been read out
                    if (ok && n >= 2) ok = mbar_wait(&bars[bOfree + b], ((n >> 1) - 1) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t tbuf = tb + b * kBufCols;
                    const uint32_t lQ = desc_lo(dK) + (smem_u32(smem + s * kStageBytes) >> 4);
                    const uint32_t lK = lQ + (kQBytes >> 4);
                    mma_ss_w<false>(lead, tbuf + colS, lQ, desc_hi(dK), lK, desc_hi(dK), iS);
#pragma unroll
                    for (int k = 1; k < kHD / 16; ++k)
                        mma_ss_w<true>(lead, tbuf + colS, lQ + k * 2, desc_hi(dK), lK + k * 2, desc_hi(dK), iS);
                    mma_commit_w(lead, &bars[bS + b]);
                    if (n >= 1) {
                        ok = mbar_wait(&bars[bP + (b ^ 1)], ((n - 1) >> 1) & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv(n - 1);
                    }
                }
                if (ok && ntiles >= 1) {
                    const int n = ntiles - 1;
                    ok = mbar_wait(&bars[bP + (n & 1)], (n >> 1) & 1, abort_flag);
                    if (ok) {
                        tc_fence_after();
                        issue_pv(n);
                    }
                }
            } else {
                // tile n: its own rows in slot (n + 1) % 4, the 128 rows before them in slot n % 4
                constexpr uint32_t iS128 = make_idesc_bf16(kQT, 128, 0, 0);
                auto slot_lo = [&](int m, uint32_t off) -> uint32_t {
                    return desc_lo(dK) + (smem_u32(smem + (m % kStages) * kStageBytes + off) >> 4);
                };
                auto issue_pv = [&](int n) {
                    const uint32_t tbuf = tb + (n & 1) * kBufCols;
                    const uint32_t lV0 = slot_lo(n, kQBytes + kKVBytes), lV1 = slot_lo(n + 1, kQBytes + kKVBytes);
                    // a head's first tile has no rows before it: their weights are zero, and the slot holds another
                    // head's rows, so those products are left out
                    const bool head_start = tile_of(n) % p.tiles_per_head == 0;
                    if (!head_start) {
                        mma_ts_w<false>(lead, tbuf + colO, tbuf + colS, lV0, desc_hi(dK), iO);
#pragma unroll
                        for (int k = 1; k < 8; ++k)
                            mma_ts_w<true>(lead, tbuf + colO, tbuf + colS + k * 8, lV0 + k * (2048 >> 4), desc_hi(dK), iO);
                        mma_ts_w<true>(lead, tbuf + colO, tbuf + colS + 64, lV1, desc_hi(dK), iO);
                    } else {
                        mma_ts_w<false>(lead, tbuf + colO, tbuf + colS + 64, lV1, desc_hi(dK), iO);
                    }
#pragma unroll
                    for (int k = 1; k < 8; ++k)
                        mma_ts_w<true>(lead, tbuf + colO, tbuf + colS + 64 + k * 8, lV1 + k * (2048 >> 4), desc_hi(dK), iO);
                    mma_commit_w(lead, &bars[bO + (n & 1)]);
                    mma_commit_w(lead, &bars[bEmpty + n % kStages]);     // the rows before tile n are dead now
                };
                if (ntiles > 0) ok = mbar_wait(&bars[bFull + 0], 0, abort_flag);       // rows before the first tile
                for (int n = 0; n < ntiles && ok; ++n) {
                    const int m = n + 1, b = n & 1;
                    ok = mbar_wait(&bars[bFull + m % kStages], (m / kStages) & 1, abort_flag);
                    if (ok && n >= 2) ok = mbar_wait(&bars[bOfree + b], ((n >> 1) - 1) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t tbuf = tb + b * kBufCols;
                    const uint32_t lQ = slot_lo(m, 0), lK0 = slot_lo(n, kQBytes), lK1 = slot_lo(m, kQBytes);
                    mma_ss_w<false>(lead, tbuf + colS, lQ, desc_hi(dK), lK0, desc_hi(dK), iS128);
                    mma_ss_w<false>(lead, tbuf + colS + 128, lQ, desc_hi(dK), lK1, desc_hi(dK), iS128);
#pragma unroll
                    for (int k = 1; k < kHD / 16; ++k) {
                        mma_ss_w<true>(lead, tbuf + colS, lQ + k * 2, desc_hi(dK), lK0 + k * 2, desc_hi(dK), iS128);
                        mma_ss_w<true>(lead, tbuf + colS + 128, lQ + k * 2, desc_hi(dK), lK1 + k * 2, desc_hi(dK), iS128);
                    }
                    mma_commit_w(lead, &bars[bS + b]);
                    if (n >= 1) {
                        ok = mbar_wait(&bars[bP + (b ^ 1)], ((n - 1) >> 1) & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv(n - 1);
                    }
                }
                if (ok && ntiles >= 1) {
                    const int n = ntiles - 1;
                    ok = mbar_wait(&bars[bP + (n & 1)], (n >> 1) & 1, abort_flag);
                    if (ok) {
                        tc_fence_after();
                        issue_pv(n);
                    }
                }
            }
        }
    } else {
        // ---- softmax groups: thread = query row r of the tile, TMEM lane r
        const int g = warp >> 2;                     // group 0: warps 0-3, group 1: warps 4-7
        const int wq = warp & 3;                     // lane quarter
        const int r = tid & 127;
        const uint32_t lane_base = (uint32_t)wq * 32u;
        const int c0 = wq * 32;                      // first score column this warp reads (PAD + 32 columns from here)
        uint8_t* ostage = smem + offOut + g * kQBytes;
        uint8_t* orow = ostage + (r >> 3) * 1024 + (r & 7) * 128;
        const uint32_t sw = r & 7;
        const uint32_t tbuf = tb + g * kBufCols;
        for (int n = g; n < ntiles && ok; n += 2) {
            const uint32_t ph = (n >> 1) & 1;
            const int tile = tile_of(n);
            const int head = tile / p.tiles_per_head, i0 = (tile % p.tiles_per_head) * kQT;
            // visible columns of this row inside its warp's batch of PAD + 32 columns: keys i-w+1 .. i, and key >= 0
            const int jhi = lane + kPad;
            int jlo = lane + kPad + 1 - p.window;
            jlo = max(jlo, kPad - i0 - c0);          // key index i0 - PAD + c0 + j must not be negative
            auto mask_word = [&](int base) -> uint32_t {
                const int a = max(jlo - base, 0), b = min(jhi - base, 31);
                if (a > b) return 0u;
                return (b - a == 31) ? 0xffffffffu : (((1u << (b - a + 1)) - 1u) << a);
            };
            float inv_l;
            if constexpr (PAD == 64) {
                const uint32_t mk[3] = {mask_word(0), mask_word(32), mask_word(64)};

                ok = group_all(1 + g, mbar_wait(&bars[bS + g], ph, abort_flag));
                if (!ok) break;
                tc_fence_after();
                {
                    uint32_t s[96];
                    {
                        uint32_t t0[32], t1[32], t2[32];
                        tmem_ld32(tmem_addr(tbuf, lane_base, colS + c0), t0);
                        tmem_ld32(tmem_addr(tbuf, lane_base, colS + c0 + 32), t1);
                        tmem_ld32(tmem_addr(tbuf, lane_base, colS + c0 + 64), t2);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) { s[i] = t0[i]; s[32 + i] = t1[i]; s[64 + i] = t2[i]; }
                    }
                    float mx = -INFINITY;
#pragma unroll
                    for (int j = 0; j < 96; ++j) {
                        const bool v = (mk[j >> 5] >> (j & 31)) & 1u;
                        const float x = v ? __uint_as_float(s[j]) : -INFINITY;
                        s[j] = __float_as_uint(x);
                        mx = fmaxf(mx, x);
                    }
                    const float mc = mx * p.scale_log2e;     // every row sees at least its own key, so mx is finite
                    float l = 0.f;
                    uint32_t pk[48];
#pragma unroll
                    for (int j = 0; j < 48; ++j) {
                        const float e0 = ex2(fmaf(__uint_as_float(s[2 * j]), p.scale_log2e, -mc));
                        const float e1 = ex2(fmaf(__uint_as_float(s[2 * j + 1]), p.scale_log2e, -mc));
                        l += e0 + e1;
                        pk[j] = pack2(e0, e1);
                    }
                    inv_l = 1.0f / l;
                    // P row: 192 keys = 96 packed columns; this warp's batch sits at packed columns [16 wq, 16 wq + 48)
                    uint32_t zero[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) zero[i] = 0u;
#pragma unroll
                    for (int gg = 0; gg < 6; ++gg)
                        if (gg < wq || gg > wq + 2) tmem_st16(tmem_addr(tbuf, lane_base, colS + gg * 16), zero);
                    uint32_t d0[16], d1[16], d2[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) { d0[i] = pk[i]; d1[i] = pk[16 + i]; d2[i] = pk[32 + i]; }
                    tmem_st16(tmem_addr(tbuf, lane_base, colS + wq * 16), d0);
                    tmem_st16(tmem_addr(tbuf, lane_base, colS + wq * 16 + 16), d1);
                    tmem_st16(tmem_addr(tbuf, lane_base, colS + wq * 16 + 32), d2);
                }
            } else {
                // 160 columns per row: two passes of five 32-column loads (maximum, then weights); the packed
                // weights of a block go over columns that this row has read already
                ok = group_all(1 + g, mbar_wait(&bars[bS + g], ph, abort_flag));
                if (!ok) break;
                tc_fence_after();
                float mx = -INFINITY;
#pragma unroll 1
                for (int b = 0; b < 5; ++b) {
                    uint32_t t[32];
                    tmem_ld32(tmem_addr(tbuf, lane_base, colS + c0 + 32 * b), t);
                    tmem_wait_ld();
                    const uint32_t m = mask_word(32 * b);
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if ((m >> i) & 1u) mx = fmaxf(mx, __uint_as_float(t[i]));
                }
                const float mc = mx * p.scale_log2e;     // every row sees at least its own key, so mx is finite
                float l = 0.f;
#pragma unroll 1
                for (int b = 0; b < 5; ++b) {
                    uint32_t t[32], pk[16];
                    tmem_ld32(tmem_addr(tbuf, lane_base, colS + c0 + 32 * b), t);
                    tmem_wait_ld();
                    const uint32_t m = mask_word(32 * b);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float x0 = ((m >> (2 * j)) & 1u) ? __uint_as_float(t[2 * j]) : -INFINITY;
                        const float x1 = ((m >> (2 * j + 1)) & 1u) ? __uint_as_float(t[2 * j + 1]) : -INFINITY;
                        const float e0 = ex2(fmaf(x0, p.scale_log2e, -mc));
                        const float e1 = ex2(fmaf(x1, p.scale_log2e, -mc));
                        l += e0 + e1;
                        pk[j] = pack2(e0, e1);
                    }
                    tmem_st16(tmem_addr(tbuf, lane_base, colS + wq * 16 + b * 16), pk);
                }
                inv_l = 1.0f / l;
                // P row: 256 keys = 128 packed columns; this warp's batch sits at packed columns [16 wq, 16 wq + 80)
                uint32_t zero[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) zero[i] = 0u;
#pragma unroll
                for (int gg = 0; gg < 8; ++gg)
                    if (gg < wq || gg > wq + 4) tmem_st16(tmem_addr(tbuf, lane_base, colS + gg * 16), zero);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&bars[bP + g]);
            ok = group_all(1 + g, mbar_wait(&bars[bO + g], ph, abort_flag));
            if (!ok) break;
            tc_fence_after();
            uint32_t o0[32], o1[32];
            tmem_ld32(tmem_addr(tbuf, lane_base, colO), o0);
            tmem_ld32(tmem_addr(tbuf, lane_base, colO + 32), o1);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(&bars[bOfree + g]);              // the TMEM buffer may take the group's next tile
            if ((tid & 127) == 0) tma_store_wait_read<0>();   // the previous store has read the staging tile
            group_sync(1 + g);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint4 v4;
                v4.x = pack2(__uint_as_float(o0[8 * j + 0]) * inv_l, __uint_as_float(o0[8 * j + 1]) * inv_l);
                v4.y = pack2(__uint_as_float(o0[8 * j + 2]) * inv_l, __uint_as_float(o0[8 * j + 3]) * inv_l);
                v4.z = pack2(__uint_as_float(o0[8 * j + 4]) * inv_l, __uint_as_float(o0[8 * j + 5]) * inv_l);
                v4.w = pack2(__uint_as_float(o0[8 * j + 6]) * inv_l, __uint_as_float(o0[8 * j + 7]) * inv_l);
                *reinterpret_cast<uint4*>(orow + ((j ^ sw) << 4)) = v4;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint4 v4;
                v4.x = pack2(__uint_as_float(o1[8 * j + 0]) * inv_l, __uint_as_float(o1[8 * j + 1]) * inv_l);
                v4.y = pack2(__uint_as_float(o1[8 * j + 2]) * inv_l, __uint_as_float(o1[8 * j + 3]) * inv_l);
                v4.z = pack2(__uint_as_float(o1[8 * j + 4]) * inv_l, __uint_as_float(o1[8 * j + 5]) * inv_l);
                v4.w = pack2(__uint_as_float(o1[8 * j + 6]) * inv_l, __uint_as_float(o1[8 * j + 7]) * inv_l);
                *reinterpret_cast<uint4*>(orow + (((4 + j) ^ sw) << 4)) = v4;
            }
            fence_proxy_async_smem();
            group_sync(1 + g);
            if ((tid & 127) == 0) {
                tma_store_3d(&tm_o, ostage, 0, i0, head);        // rows past the sequence end are clipped
                tma_store_commit();
            }
        }
        if ((tid & 127) == 0) tma_store_wait<0>();
    }

    if (!ok && lane == 0) atomicOr(p.err, 1u);
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int it = 0; it < 200; ++it) __nanosleep(1000);
    }
    __syncthreads();
    if (warp == kWarpMma) tmem_dealloc(tb, 512);
}

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool make_map(CUtensorMap* m, const void* base, int BH, int L, int box_rows) {
    static EncodeTiledFn enc = nullptr;
    if (!enc) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return false;
        enc = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    cuuint64_t dims[3] = {(cuuint64_t)kHD, (cuuint64_t)L, (cuuint64_t)BH};
    cuuint64_t strides[2] = {(cuuint64_t)kHD * 2, (cuuint64_t)L * kHD * 2};
    cuuint32_t box[3] = {(cuuint32_t)kHD, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool swa_tc_supported(int window) { return window >= 1 && window <= 128; }

template <int PAD>
static based_status launch_swa_pad(const void* q, const void* k, const void* v, void* out, int BH, int L, int window,
                                   float scale, cudaStream_t stream) {
    using C = SwaCfg<PAD>;
    CUtensorMap tq, tk, tv, to;
    constexpr int kv_rows = PAD == 64 ? C::kKeys : kQT;      // rows of one K / V load
    if (!make_map(&tq, q, BH, L, kQT) || !make_map(&tk, k, BH, L, kv_rows) || !make_map(&tv, v, BH, L, kv_rows) ||
        !make_map(&to, out, BH, L, kQT))
        return BASED_ERR_CUDA;
    SwaParams p;
    if (error_word_ptr(&p.err) != BASED_OK) return BASED_ERR_CUDA;
    p.L = L;
    p.window = window;
    p.tiles_per_head = (L + kQT - 1) / kQT;
    p.total_tiles = p.tiles_per_head * BH;
    p.scale_log2e = scale * 1.4426950408889634f;
    static int sm_count[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BASED_ERR_CUDA;
    {
        std::lock_guard<std::mutex> lock(setup_mutex());
        if (sm_count[dev] == 0) {
            if (cudaFuncSetAttribute(swa_tc_kernel<PAD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)C::kSmemBytes) != cudaSuccess)
                return BASED_ERR_CUDA;
            int n = 148;
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
            sm_count[dev] = n > 0 ? n : 148;
        }
    }
    const int sms = sm_count[dev];
    const int grid = p.total_tiles < sms ? p.total_tiles : sms;
    swa_tc_kernel<PAD><<<grid, kThreads, C::kSmemBytes, stream>>>(tq, tk, tv, to, p);
    note_launch();
    return check_launch("swa_tc_kernel");
}

based_status launch_swa_tc(const void* q, const void* k, const void* v, void* out, int BH, int L, int window,
                           float scale, cudaStream_t stream) {
    if (window <= 64) return launch_swa_pad<64>(q, k, v, out, BH, L, window, scale, stream);
    return launch_swa_pad<128>(q, k, v, out, BH, L, window, scale, stream);
}

}  // namespace based
