// based_prefill_backward, bf16 tensor-core path (tcgen05 / TMEM / TMA): the same three passes as
// the fp32 path (row statistics, dq, dk + dv; see backward_simt.cu for the formulas), with every
// 128 x 128 tile of (query, key) pairs evaluated by tensor-core products:
//
//   S  = Q_i K_j^T          (K = 16)          GV = G_i V_j^T   (K = d_v; G = dout, exact in bf16)
//   dq:   DS = (GV / D_i + b_i)(1/4 + S/16) [j<=i]  as bf16 in tensor memory,   dQ_i += DS K_j
//   dk/dv: the transposed products S^T = K_j Q_i^T, GV^T = V_j G_i^T;  W'^T = w(S^T) / D_i and DS^T in
//          tensor memory (over the scores, in place);   dV_j += W'^T G_i,   dK_j += DS^T Q_i
// 1/D_i is applied to the fp32 products, not to the operand: a = dout / D rounded to bf16 would
// break the near-cancellation of a_i.v_j + b_i for short prefixes.
//
// When the caller passes the forward output, statistics and dq take one sweep (a fifth mode):
//   dq_i = X_i / D_i + (m_i / D_i + b_i) Y_i,   X_i = sum_j w'_ij (gv_ij - m_i) k_j,   Y_i = sum_j w'_ij k_j
// holds for any m_i and needs neither D_i nor b_i while the keys are swept: D_i and E_i accumulate in
// registers, X and Y by MMA from two packed bf16 tiles, and 1/D_i, b_i, dq_i are formed in fp32 at the
// end.  m_i = dout_i . out_i is the weighted mean E_i / D_i of the gv_ij up to the rounding of out, so
// the packed products are as small as ds above and the part of dq that cancels against b_i stays in
// fp32 (without a centre the two separately rounded tiles would have to cancel).
//
// One CTA per (head, 128-row tile), 160 threads: warps 0-3 own one accumulator row each (the
// polynomial, masks and bf16 packing), warp 4 issues TMA loads and MMAs (converged, one elected lane).  The loop over
// the other side's tiles is sequential per CTA (loads of the next tile are in flight during the
// current one); parallelism comes from the (tile, head) grid.  q and k tiles are loaded 32
// columns wide (columns 16..31 are zero-filled by TMA) so that they serve both as K-major
// operands of the scores and as MN-major B operands of dQ / dK.  The work is O(L^2) per head, as
// in the fp32 path.  A fourth mode of the same kernel evaluates the forward pass in this form
// (scores, weights as bf16 in tensor memory, Y += P V, row sums): the tensor-core path of the
// feature dimensions 8, 24 and 32, which the chunked d' = 16 kernel does not cover.  All modes take
// d' (8, 16, 24, 32) as a parameter: the polynomial's coefficients 1/sqrt(d'), 1/(2 d'), a second K
// step of the scores above 16, and up to 32 gradient columns of dq and dk.
//
// Block-wise path (template flag XB; d' = 16, statistics in one sweep): linear in L.  The loops of the merged
// statistics + dq pass and of the dk/dv pass stop at the edges of the own tile's block of W tokens; all earlier
// blocks reach a query, and all later blocks a key, through one state tile each (block_state_tc.cu writes them:
// S = sum mono(k) v^T with row sums z for the queries, R = sum mono(q) (dout / D)^T with row sums R_b = sum b mono(q)
// for the keys, in the basis of the 153 distinct monomials of the feature map).  Before its loop such a CTA
// multiplies its own wide tile with the state tile (T = G S^T or V R^T, 128 x 160 in tensor memory), every row
// thread contracts its row of T with the monomials and the Jacobian of its q or k row, and the results start the
// accumulators that the loop's products add to; the dk/dv pass also writes the monomials of its k rows back to
// tensor memory as the A operand of dV = mono(K) R.
#include <math.h>

#include <mutex>
#include <type_traits>

#include "common.cuh"
#include "sm100.cuh"

namespace based {
using namespace sm100;

namespace {
constexpr int kTile = 128;
constexpr int kThreadsB = 160;
constexpr int kModeStats = 0, kModeDq = 1, kModeDkDv = 2, kModeFwd = 3, kModeDqS = 4;
constexpr uint32_t kQKTile = kTile * 64;                 // [128][32] bf16, 64-byte rows, SWIZZLE_64B

// LT: rows of the tiles the CTA loops over (columns of the accumulators): 64 where that lets two CTAs
// share an SM (256 tensor-memory columns each), so that one CTA's row-thread pass overlaps the
// other's MMA bursts; 128 for the dk/dv pass at d_v 128, whose accumulators need more columns.
template <int DV, int MODE, int LT, bool XB = false> struct BCfg {
    static constexpr int kVB = (DV + 63) / 64;           // 64-column blocks of a [rows][DV] tile (112 -> 2, second partly zero)
    static constexpr uint32_t kWide = kVB * kTile * 128; // own tile: [128][64 * kVB] bf16 in SWIZZLE_128B blocks
    static constexpr uint32_t kNarrowL = LT * 64, kWideL = kVB * LT * 128;       // looped tiles
    // shared memory: resident narrow + wide tile, two stages of (narrow + wide), (1/D, b) of two stages, barriers
    static constexpr uint32_t offResN = 0, offResW = offResN + kQKTile;
    static constexpr uint32_t offStage = offResW + kWide, kStage = kNarrowL + kWideL;
    // a block state, transposed: [64 * kVB value columns][160 features] bf16 in five SWIZZLE_64B blocks of 32 features
    // (block-wise path); it lies from the second stage on, so that the first looped tile loads beside it
    static constexpr uint32_t kStateBlk = kVB * 64 * 64;
    static constexpr uint32_t kStateTile = 5 * kStateBlk;
    static constexpr uint32_t kStageArea = (XB && kStage + kStateTile > 2 * kStage) ? kStage + kStateTile : 2 * kStage;
    static constexpr uint32_t offB = offStage + kStageArea;
    static constexpr uint32_t offMisc = offB + 2 * LT * 8;
    static constexpr uint32_t kSmem = offMisc + 2048 + 1024;                    // barriers, the block state's row sums (160 floats), m (128)

    // tensor memory columns: scores, dout.v products, ds (dq pass; the dk/dv pass packs in place), accumulators
    static constexpr uint32_t colS = 0, colG = LT, colD = MODE == kModeFwd ? LT : 2 * LT;   // forward: no dout.v product
    static constexpr uint32_t colD2 = colD + LT / 2;                                      // second packed tile (merged pass)
    static constexpr uint32_t colAcc = MODE == kModeDq ? 2 * LT + LT / 2                  // dQ (32)
                                       : MODE == kModeDqS ? 3 * LT                        // X (32), then Y (32)
                                       : MODE == kModeFwd ? LT + LT / 2                   // Y (64 * kVB)
                                                          : (LT == 32 ? 96 : 2 * LT < 160 ? 160 : 2 * LT);  // dV (64 * kVB): above the block
                                       // product (160 columns), or with 32-row looped tiles above its packed monomials (80): the
                                       // product is read before the first dV product is issued
    static constexpr uint32_t colAcc2 = colAcc + 32;                                      // merged pass: Y
    static constexpr uint32_t colK = colAcc + 64 * kVB;                                   // dK (32), dk/dv pass
    static constexpr uint32_t kColsUsed = MODE == kModeStats ? 2 * LT
                                          : MODE == kModeDq ? colAcc + 32
                                          : MODE == kModeDqS ? colAcc2 + 32
                                          : MODE == kModeFwd ? colAcc + 64 * kVB
                                                             : colK + 32;
    static constexpr uint32_t kCols = kColsUsed <= 128 ? 128 : kColsUsed <= 256 ? 256 : 512;
    static_assert(kColsUsed <= 512, "tensor memory budget");
};
enum { bRes = 0, bFull0, bFull1, bMma, bAlu, bFinal, bXs, bX0, bX1, bNum };

struct BParams {
    const __nv_bfloat16* g_raw;  // dout and the forward output as plain pointers [BH, L, dvw] (merged pass)
    const __nv_bfloat16* o_raw;
    const float2* stats_in;      // (1/D, b) per row (dq, dk/dv passes)
    float2* stats_out;           // statistics pass
    __nv_bfloat16* dq;           // [BH, L, 16]
    __nv_bfloat16* dk;
    __nv_bfloat16* dvo;          // [BH, L, dvw]
    unsigned int* err;
    int L, dvw, numerator_only;  // dvw: value head dimension of the caller's tensors (64, 112, 128)
    int df, kdim;                // feature dimension d', and d' rounded up to 16 (K extent of the scores)
    float s1, s2;                // w = 1 + s * s1 + s^2 * s2 (1 / sqrt d', 1 / (2 d'))
    // block-wise path: pairs inside a block of W tokens by tiles, the other blocks through their summed state
    int W, nblk;
    const float* sv;             // [BH x nblk][160]: row sums of the block states (z, or the b-weighted sums of phi(q))
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// AND of a predicate over the 128 row threads (named barrier 1): all of them get the same answer, so
// they leave their loop together and the warp-collective tensor-memory accesses stay converged; it
// also orders their shared-memory writes before the reads that follow
__device__ __forceinline__ bool rows_all(bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 1, 128, p;\n\t"
        "selp.b32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred)
        : "memory");
    return r != 0;
}
// w = 1 + s / sqrt(d') + s^2 / (2 d') and its derivative, s1 = 1 / sqrt(d'), s2 = 1 / (2 d') (d' = 16: 1/4, 1/32)
__device__ __forceinline__ float tw(float s, float s1, float s2) { return fmaf(s, fmaf(s, s2, s1), 1.0f); }
__device__ __forceinline__ float tdw(float s, float s1, float s2) { return fmaf(s, 2.0f * s2, s1); }

// Block-wise path, one row thread: T (160 fp32 columns of tensor memory, from column 0) holds the product of the
// row's wide operand with a block state in the monomial basis of block_state_tc_kernel
// (f < 16: x_f | 16 + 16 o + m: x_m x_(m+o) | 144 + m: x_m x_(m+8) | 152: 1), sv the state's row sums.
//   query row (merged statistics + dq pass): T_f = (S g_i)_f, sv = z:
//     den += mono(q_i) . z,  en += mono(q_i) . T,  gx = J^T (T - m_i z),  gy = J^T z      (J = d mono / d q_i)
//   key row (dk/dv pass): T_f = (R v_j)_f, sv = R_b:  gx = J^T (T + R_b); the monomials of k_j go back to tensor
//     memory as packed bf16 (80 columns from column 0, over the columns already read): the A operand of dV += mono(K) R
template <bool KEYS>
__device__ __forceinline__ void block_rows(uint32_t tb, uint32_t lane_base, const float (&x)[16], const float* sv,
                                           float m_own, float& den, float& en, float (&gx)[16], float (&gy)[16]) {
#pragma unroll
    for (int blk = 0; blk < 5; ++blk) {
        uint32_t tr[32];
        tmem_ld32(tmem_addr(tb, lane_base, blk * 32), tr);
        tmem_wait_ld();
        float mono[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int f = blk * 32 + i;
            const int m = f < 16 ? f : f < 144 ? ((f - 16) & 15) : f < 152 ? f - 144 : -1;
            const int n = f < 16 ? -1 : f < 144 ? ((m + ((f - 16) >> 4)) & 15) : f < 152 ? m + 8 : -1;
            mono[i] = 0.f;
            if (f <= 152) {
                const float xm = m >= 0 ? x[m] : 1.0f, xn = n >= 0 ? x[n] : 1.0f;
                mono[i] = xm * xn;
                const float a = __uint_as_float(tr[i]), zf = sv[f];
                const float bq = KEYS ? a + zf : fmaf(-m_own, zf, a);
                if (!KEYS) {
                    den = fmaf(mono[i], zf, den);
                    en = fmaf(mono[i], a, en);
                }
                if (m >= 0 && n < 0) {
                    gx[m] += bq;
                    if (!KEYS) gy[m] += zf;
                } else if (m >= 0 && m != n) {
                    gx[m] = fmaf(xn, bq, gx[m]);
                    gx[n] = fmaf(xm, bq, gx[n]);
                    if (!KEYS) { gy[m] = fmaf(xn, zf, gy[m]); gy[n] = fmaf(xm, zf, gy[n]); }
                } else if (m >= 0) {
                    gx[m] = fmaf(2.0f * xm, bq, gx[m]);
                    if (!KEYS) gy[m] = fmaf(2.0f * xm, zf, gy[m]);
                }
            }
        }
        if (KEYS) {
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = pack_bf16x2(mono[2 * i], mono[2 * i + 1]);
            tmem_st16(tmem_addr(tb, lane_base, blk * 16), pk);
        }
    }
}
}  // namespace

// tm_n0 / tm_w0: narrow (q or k) and wide (a/g or v) tensor of the CTA's own (resident) tile;
// tm_n1 / tm_w1: of the tiles it loops over.
// XB: the block-wise path (merged statistics + dq pass and dk/dv pass, d' = 16); tm_st: the block states,
// transposed: [BH x nblk][d_v][160] bf16.  tm_out: the wide output (dv, or the forward output), stored by TMA.
template <int DV, int MODE, int LT, bool XB>
__global__ void __launch_bounds__(kThreadsB, 1)
    backward_tc_kernel(const __grid_constant__ CUtensorMap tm_n0, const __grid_constant__ CUtensorMap tm_w0,
                       const __grid_constant__ CUtensorMap tm_n1, const __grid_constant__ CUtensorMap tm_w1,
                       const __grid_constant__ CUtensorMap tm_st, const __grid_constant__ CUtensorMap tm_out,
                       const BParams p) {
    static_assert(!XB || MODE == kModeDqS || MODE == kModeDkDv, "block-wise path: the two passes that use it");
    using C = BCfg<DV, MODE, LT, XB>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::offMisc);
    uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(bars + bNum);
    volatile uint32_t* abort_flag = tmem_base_s + 1;
    float2* s_b = reinterpret_cast<float2*>(smem + C::offB);
    float* s_sv = reinterpret_cast<float*>(smem + C::offMisc + 256);
    float* s_m = reinterpret_cast<float*>(smem + C::offMisc + 1024);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ntiles = (p.L + kTile - 1) / kTile;
    // own tile: the longest loops first (dq, statistics: last query tiles; dk/dv: first key tiles)
    const int own = MODE == kModeDkDv ? blockIdx.x : ntiles - 1 - blockIdx.x;
    const int head = blockIdx.y;
    const int r0 = own * kTile;
    // looped tiles (LT rows each): keys 0 .. end of the own tile, or queries from the own tile's first row on
    // block-wise path: the loop stays inside the own tile's block of W tokens; the blocks before it (queries) or
    // after it (keys) enter through their summed state, if there are any (cross)
    const int blk = XB ? r0 / p.W : 0;
    const bool cross = XB && (MODE == kModeDkDv ? blk + 1 < p.nblk : blk > 0);
    const int first = MODE == kModeDkDv ? r0 / LT : (XB ? blk * p.W / LT : 0);
    const int last = MODE == kModeDkDv ? (min(p.L, XB ? (blk + 1) * p.W : p.L) - 1) / LT : (min(p.L, r0 + kTile) - 1) / LT;
    const int nloop = last - first + 1;

    if (tid == 0) {
        mbar_init(&bars[bRes], 1); mbar_init(&bars[bFull0], 1); mbar_init(&bars[bFull1], 1);
        mbar_init(&bars[bMma], 1); mbar_init(&bars[bAlu], 128); mbar_init(&bars[bFinal], 1);
        mbar_init(&bars[bXs], 1); mbar_init(&bars[bX0], 1); mbar_init(&bars[bX1], 128);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 4) { tmem_alloc(tmem_base_s, C::kCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = *tmem_base_s;
    bool ok = true;

    // descriptors: narrow tiles (64-byte rows, SWIZZLE_64B), wide tiles (128-byte rows, SWIZZLE_128B, 64-column blocks)
    constexpr uint64_t dN = make_smem_desc_base(16, 512, kSwizzle64B);                  // K-major, or MN-major one block
    constexpr uint64_t dW = make_smem_desc_base(kTile * 128, 1024, kSwizzle128B);       // own wide tile (128 rows per block)
    constexpr uint64_t dWL = make_smem_desc_base(LT * 128, 1024, kSwizzle128B);         // looped wide tile (LT rows per block)
    constexpr uint32_t iS = make_idesc_bf16(128, LT, 0, 0);                             // both operands K-major
    constexpr uint32_t iN32 = make_idesc_bf16(128, 32, 0, 1);                           // A from TMEM, B MN-major narrow
    constexpr uint32_t iNV = make_idesc_bf16(128, 64 * C::kVB, 0, 1);                   // A from TMEM, B MN-major wide
    constexpr uint64_t dStN = make_smem_desc_base(C::kStateBlk, 512, kSwizzle64B);      // block state as B over d_v: MN-major
    constexpr uint32_t iT = make_idesc_bf16(128, 160, 0, 1);                            // own wide x state^T
    constexpr uint32_t iXV = make_idesc_bf16(128, 64 * C::kVB, 0, 0);                   // A from TMEM, B K-major: the state over features

    if (warp == 4) {
        {
            // the whole warp runs this block; one elected lane issues the MMAs, commits and loads (see mma_ss_w)
            const uint32_t lead = elect_one();
            const uint32_t aResN = smem_u32(smem + C::offResN), aResW = smem_u32(smem + C::offResW);
            auto load_stage = [&](int it) {
                if (!lead) return;
                const int s = it & 1;
                uint8_t* st = smem + C::offStage + s * C::kStage;
                const int row = (first + it) * LT;
                mbar_arrive_expect_tx(&bars[bFull0 + s], C::kStage);
                tma_load_3d(st, &tm_n1, &bars[bFull0 + s], 0, row, head);
#pragma unroll
                for (int b = 0; b < C::kVB; ++b)
                    tma_load_3d(st + C::kNarrowL + b * (LT * 128), &tm_w1, &bars[bFull0 + s], b * 64, row, head);
            };
            if (lead) {
            mbar_arrive_expect_tx(&bars[bRes], MODE == kModeFwd ? kQKTile : kQKTile + C::kWide);
            tma_load_3d(smem + C::offResN, &tm_n0, &bars[bRes], 0, r0, head);
            if (MODE != kModeFwd) {
#pragma unroll
                for (int b = 0; b < C::kVB; ++b)
                    tma_load_3d(smem + C::offResW + b * (kTile * 128), &tm_w0, &bars[bRes], b * 64, r0, head);
            }
            if (cross) {
                mbar_arrive_expect_tx(&bars[bXs], C::kStateTile);
#pragma unroll
                for (int b = 0; b < 5; ++b)
                    tma_load_3d(smem + C::offStage + C::kStage + b * C::kStateBlk, &tm_st, &bars[bXs], b * 32, 0,
                                head * p.nblk + blk);
            }
            }
            load_stage(0);
            ok = mbar_wait(&bars[bRes], 0, abort_flag);
            if (cross && ok) {
                const uint32_t aSt = smem_u32(smem + C::offStage + C::kStage);
                ok = mbar_wait(&bars[bXs], 0, abort_flag);
                tc_fence_after();
                // T = own wide tile x state^T (K = d_v), 160 columns from column 0
#pragma unroll
                for (int kk = 0; kk < DV / 16; ++kk) {
                    const uint32_t off = ((kk >> 2) * (kTile * 128) + (kk & 3) * 32) >> 4;
                    const uint32_t offS = (kk * 1024) >> 4;        // sixteen value columns = sixteen 64-byte rows of every block
                    if (kk == 0)
                        mma_ss_w<false>(lead, tb, desc_lo(dW) + (aResW >> 4) + off, desc_hi(dW), desc_lo(dStN) + (aSt >> 4) + offS,
                                         desc_hi(dStN), iT);
                    else
                        mma_ss_w<true>(lead, tb, desc_lo(dW) + (aResW >> 4) + off, desc_hi(dW), desc_lo(dStN) + (aSt >> 4) + offS,
                                        desc_hi(dStN), iT);
                }
                mma_commit_w(lead, &bars[bX0]);
                if (MODE == kModeDkDv) {
                    // dV = mono(K) (tensor memory, written by the row threads) x state (K-major: 64-byte rows of 32
                    // features, 160 = 10 K-steps of 32 bytes)
                    if (ok) ok = mbar_wait(&bars[bX1], 0, abort_flag);
                    tc_fence_after();
                    if (ok) {
#pragma unroll
                        for (int k = 0; k < 10; ++k) {
                            const uint32_t offK = ((k >> 1) * C::kStateBlk + (k & 1) * 32) >> 4;
                            if (k == 0)
                                mma_ts_w<false>(lead, tb + C::colAcc, tb + k * 8, desc_lo(dN) + (aSt >> 4) + offK, desc_hi(dN), iXV);
                            else
                                mma_ts_w<true>(lead, tb + C::colAcc, tb + k * 8, desc_lo(dN) + (aSt >> 4) + offK, desc_hi(dN), iXV);
                        }
                    }
                } else {
                    if (ok) ok = mbar_wait(&bars[bX1], 0, abort_flag);     // the rows have read T: the scores may overwrite it
                    tc_fence_after();
                }
                // the state tile's stages are loaded again after the first iteration's products (in-order pipe)
            }
            for (int it = 0; it < nloop && ok; ++it) {
                const int s = it & 1;
                const uint32_t aN = smem_u32(smem + C::offStage + s * C::kStage), aW = aN + C::kNarrowL;
                ok = mbar_wait(&bars[bFull0 + s], (it >> 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                // scores: rows = own tile, columns = looped tile
                mma_ss_w<false>(lead, tb + C::colS, desc_lo(dN) + (aResN >> 4), desc_hi(dN), desc_lo(dN) + (aN >> 4),
                                 desc_hi(dN), iS);
                if (p.kdim > 16)                             // feature dimensions 24 and 32: second K-step
                    mma_ss_w<true>(lead, tb + C::colS, desc_lo(dN) + (aResN >> 4) + 2, desc_hi(dN), desc_lo(dN) + (aN >> 4) + 2,
                                    desc_hi(dN), iS);
                // own wide tile x looped wide tile^T over d_v
#pragma unroll
                for (int kk = 0; kk < (MODE == kModeFwd ? 0 : DV / 16); ++kk) {
                    const uint32_t off = ((kk >> 2) * (kTile * 128) + (kk & 3) * 32) >> 4;
                    const uint32_t offL = ((kk >> 2) * (LT * 128) + (kk & 3) * 32) >> 4;
                    if (kk == 0)
                        mma_ss_w<false>(lead, tb + C::colG, desc_lo(dW) + (aResW >> 4) + off, desc_hi(dW),
                                         desc_lo(dWL) + (aW >> 4) + offL, desc_hi(dWL), iS);
                    else
                        mma_ss_w<true>(lead, tb + C::colG, desc_lo(dW) + (aResW >> 4) + off, desc_hi(dW),
                                        desc_lo(dWL) + (aW >> 4) + offL, desc_hi(dWL), iS);
                }
                mma_commit_w(lead, &bars[bMma]);
                // once these products are done, so are the previous iteration's (in-order pipe): its stage is free
                ok = mbar_wait(&bars[bMma], it & 1, abort_flag);
                if (!ok) break;
                if (it + 1 < nloop) load_stage(it + 1);
                ok = mbar_wait(&bars[bAlu], it & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                if (MODE == kModeDq) {
                    // dQ += DS (tensor memory, LT keys = LT/16 K-steps) x K_j (MN-major, 32 columns)
#pragma unroll
                    for (int k = 0; k < LT / 16; ++k) {
                        if (it == 0 && k == 0)
                            mma_ts_w<false>(lead, tb + C::colAcc, tb + C::colD + k * 8, desc_lo(dN) + ((aN + k * 1024) >> 4),
                                             desc_hi(dN), iN32);
                        else
                            mma_ts_w<true>(lead, tb + C::colAcc, tb + C::colD + k * 8, desc_lo(dN) + ((aN + k * 1024) >> 4),
                                            desc_hi(dN), iN32);
                    }
                } else if (MODE == kModeDqS) {
                    // X += (w' (gv - m)) K_j and Y += w' K_j: two packed tiles in tensor memory, the same B operand
#pragma unroll
                    for (int k = 0; k < LT / 16; ++k) {
                        if (it == 0 && k == 0 && !cross) {
                            mma_ts_w<false>(lead, tb + C::colAcc, tb + C::colD + k * 8, desc_lo(dN) + ((aN + k * 1024) >> 4),
                                             desc_hi(dN), iN32);
                            mma_ts_w<false>(lead, tb + C::colAcc2, tb + C::colD2 + k * 8, desc_lo(dN) + ((aN + k * 1024) >> 4),
                                             desc_hi(dN), iN32);
                        } else {
                            mma_ts_w<true>(lead, tb + C::colAcc, tb + C::colD + k * 8, desc_lo(dN) + ((aN + k * 1024) >> 4),
                                            desc_hi(dN), iN32);
                            mma_ts_w<true>(lead, tb + C::colAcc2, tb + C::colD2 + k * 8, desc_lo(dN) + ((aN + k * 1024) >> 4),
                                            desc_hi(dN), iN32);
                        }
                    }
                } else if (MODE == kModeFwd) {
                    // Y += P (tensor memory) x V_j
#pragma unroll
                    for (int k = 0; k < LT / 16; ++k) {
                        if (it == 0 && k == 0)
                            mma_ts_w<false>(lead, tb + C::colAcc, tb + C::colD + k * 8, desc_lo(dWL) + ((aW + k * 2048) >> 4),
                                             desc_hi(dWL), iNV);
                        else
                            mma_ts_w<true>(lead, tb + C::colAcc, tb + C::colD + k * 8, desc_lo(dWL) + ((aW + k * 2048) >> 4),
                                            desc_hi(dWL), iNV);
                    }
                } else if (MODE == kModeDkDv) {
                    // dV += W'^T (over the scores) x G_i;  dK += DS^T (over GV) x Q_i
#pragma unroll
                    for (int k = 0; k < LT / 16; ++k) {
                        if (it == 0 && k == 0 && !cross) {
                            mma_ts_w<false>(lead, tb + C::colAcc, tb + C::colS + k * 8, desc_lo(dWL) + ((aW + k * 2048) >> 4),
                                             desc_hi(dWL), iNV);
                            mma_ts_w<false>(lead, tb + C::colK, tb + C::colG + k * 8, desc_lo(dN) + ((aN + k * 1024) >> 4),
                                             desc_hi(dN), iN32);
                        } else {
                            mma_ts_w<true>(lead, tb + C::colAcc, tb + C::colS + k * 8, desc_lo(dWL) + ((aW + k * 2048) >> 4),
                                            desc_hi(dWL), iNV);
                            mma_ts_w<true>(lead, tb + C::colK, tb + C::colG + k * 8, desc_lo(dN) + ((aN + k * 1024) >> 4),
                                            desc_hi(dN), iN32);
                        }
                    }
                }
            }
            if (ok) mma_commit_w(lead, &bars[bFinal]);
        }
    } else {
        // ===================================================================== row threads
        const int t = tid;                                   // accumulator row == TMEM lane
        const uint32_t lane_base = (uint32_t)warp * 32u;
        const int row = r0 + t;                              // query (statistics, dq) or key (dk/dv) of this thread
        float den = 0.f, en = 0.f;
        float2 st_own = make_float2(0.f, 0.f);               // (1/D, b) of this thread's query (dq pass)
        if (MODE == kModeDq && row < p.L) st_own = p.stats_in[(size_t)head * p.L + row];
        // merged pass: the products dout_i . v_j enter the packed tile relative to m_i = dout_i . out_i, which
        // is their weighted mean E_i / D_i up to the rounding of out: the part of dq that cancels against
        // b_i is then formed in fp32 at the end, not from two separately rounded bf16 tiles
        // the block state's row sums: read by the row threads only, after their next barrier
        if (XB && cross) {
            const float* svp = p.sv + ((size_t)head * p.nblk + blk) * 160;
            s_sv[t] = svp[t];
            if (t < 32) s_sv[128 + t] = svp[128 + t];
        }
        float m_own = 0.f;
        if (MODE == kModeDqS && !p.numerator_only && (DV == 64 || p.dvw == 128)) {
            // a warp's 32 rows of out lie one after the other in global memory: every load instruction takes 512
            // consecutive bytes (two rows at d_v 128, four at d_v 64); the matching piece of dout comes from the own
            // tile in shared memory, and the lanes of a row add up their parts
            constexpr int PPR = DV / 8;                       // 16-byte pieces per row
            constexpr int NI = PPR;                           // load instructions per warp: 32 rows x PPR pieces / 32 lanes
            const int wrow0 = r0 + warp * 32;
            const uint4* op = reinterpret_cast<const uint4*>(p.o_raw + ((size_t)head * p.L + wrow0) * DV);
            uint4 ob[NI];
#pragma unroll
            for (int i = 0; i < NI; ++i) {
                const int pc = i * 32 + lane;                 // piece of the warp's 32 x PPR
                ob[i] = wrow0 + pc / PPR < p.L ? op[pc] : make_uint4(0u, 0u, 0u, 0u);
            }
            ok = rows_all(mbar_wait(&bars[bRes], 0, abort_flag));
#pragma unroll
            for (int i = 0; i < NI; ++i) {
                const int pc = i * 32 + lane;
                const int rr = warp * 32 + pc / PPR, c = pc % PPR;           // row of the tile, piece of the row
                const uint4 u = *reinterpret_cast<const uint4*>(smem + C::offResW + (c >> 3) * (kTile * 128) + rr * 128 +
                                                                (((c & 7) ^ (rr & 7)) << 4));
                const __nv_bfloat162* ha = reinterpret_cast<const __nv_bfloat162*>(&u);
                const __nv_bfloat162* hb = reinterpret_cast<const __nv_bfloat162*>(&ob[i]);
                float d = 0.f;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 fa = __bfloat1622float2(ha[e]), fb = __bfloat1622float2(hb[e]);
                    d = fmaf(fa.x, fb.x, d);
                    d = fmaf(fa.y, fb.y, d);
                }
#pragma unroll
                for (int o = PPR / 2; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
                if (c == 0) s_m[rr] = d;
            }
            __syncwarp();
            m_own = s_m[t];
        } else if (MODE == kModeDqS && !p.numerator_only && row < p.L) {
            const uint4* gp = reinterpret_cast<const uint4*>(p.g_raw + ((size_t)head * p.L + row) * p.dvw);
            const uint4* op = reinterpret_cast<const uint4*>(p.o_raw + ((size_t)head * p.L + row) * p.dvw);
            float part[4] = {0.f, 0.f, 0.f, 0.f};
            for (int c0 = 0; c0 < p.dvw / 8; c0 += 4) {          // 112 columns: 14 pieces; four in flight
                uint4 a[4], b[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const bool in = c0 + u < p.dvw / 8;
                    a[u] = in ? gp[c0 + u] : make_uint4(0u, 0u, 0u, 0u);
                    b[u] = in ? op[c0 + u] : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const __nv_bfloat162* ha = reinterpret_cast<const __nv_bfloat162*>(&a[u]);
                    const __nv_bfloat162* hb = reinterpret_cast<const __nv_bfloat162*>(&b[u]);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 fa = __bfloat1622float2(ha[e]), fb = __bfloat1622float2(hb[e]);
                        part[u] = fmaf(fa.x, fb.x, part[u]);
                        part[u] = fmaf(fa.y, fb.y, part[u]);
                    }
                }
            }
            m_own = (part[0] + part[1]) + (part[2] + part[3]);
        }
        if (XB && cross) {
            // the blocks before (queries) or after (keys) the own one, through their summed state
            ok = rows_all(mbar_wait(&bars[bRes], 0, abort_flag) && mbar_wait(&bars[bX0], 0, abort_flag));
            tc_fence_after();
            if (ok) {
                // this thread's q or k row: 64-byte rows, SWIZZLE_64B (16-byte pieces 0 and 1)
                float x[16], gx[16], gy[16];
                const uint8_t* xrow = smem + C::offResN + t * 64;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const uint4 u = *reinterpret_cast<const uint4*>(xrow + ((c ^ ((t >> 1) & 3)) << 4));
                    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float2 fv = __bfloat1622float2(h[i]);
                        x[c * 8 + 2 * i] = fv.x;
                        x[c * 8 + 2 * i + 1] = fv.y;
                    }
                }
#pragma unroll
                for (int i = 0; i < 16; ++i) { gx[i] = 0.f; gy[i] = 0.f; }
                block_rows<MODE == kModeDkDv>(tb, lane_base, x, s_sv, m_own, den, en, gx, gy);
                // the sums start the accumulators that the loop's products add to: X and Y, or dK
                uint32_t o[16], zero[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) { o[i] = __float_as_uint(gx[i]); zero[i] = 0u; }
                tmem_st16(tmem_addr(tb, lane_base, MODE == kModeDkDv ? C::colK : C::colAcc), o);
                tmem_st16(tmem_addr(tb, lane_base, (MODE == kModeDkDv ? C::colK : C::colAcc) + 16), zero);
                if (MODE == kModeDqS) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(gy[i]);
                    tmem_st16(tmem_addr(tb, lane_base, C::colAcc2), o);
                    tmem_st16(tmem_addr(tb, lane_base, C::colAcc2 + 16), zero);
                }
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(&bars[bX1]);
            }
        }
        for (int it = 0; it < nloop && ok; ++it) {
            const int c0 = (first + it) * LT;                // first row of the looped tile (columns of the accumulators)
            if (MODE == kModeDkDv && t < LT)                 // (1/D, b) of the looped queries
                s_b[(it & 1) * LT + t] = c0 + t < p.L ? p.stats_in[(size_t)head * p.L + c0 + t] : make_float2(0.f, 0.f);
            ok = rows_all(mbar_wait(&bars[bMma], it & 1, abort_flag));
            if (!ok) break;
            tc_fence_after();
            // one pass over the tile's LT accumulator columns of this row; MASKED: the tile touches the
            // diagonal or the end of the sequence (the others need no per-pair test)
            auto pass = [&](auto masked_tag) {
                constexpr bool MASKED = decltype(masked_tag)::value;
#pragma unroll 1
                for (int blk = 0; blk < LT / 32; ++blk) {
                    uint32_t sr[32], gr[32];
                    tmem_ld32(tmem_addr(tb, lane_base, C::colS + blk * 32), sr);
                    if (MODE != kModeFwd) tmem_ld32(tmem_addr(tb, lane_base, C::colG + blk * 32), gr);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int col = c0 + blk * 32 + i;
                        const float s = __uint_as_float(sr[i]), gvv = MODE == kModeFwd ? 0.f : __uint_as_float(gr[i]);
                        // pair (query, key): own row is the query except in the dk/dv pass
                        const bool live = !MASKED || (MODE == kModeDkDv ? (row <= col && col < p.L) : (col <= row));
                        float w = live ? tw(s, p.s1, p.s2) : 0.f;
                        float ds = 0.f;
                        if (MODE == kModeFwd) {
                            den += w;
                        } else if (MODE == kModeStats) {
                            den += w;
                            en = fmaf(w, gvv, en);
                        } else if (MODE == kModeDqS) {
                            den += w;
                            en = fmaf(w, gvv, en);
                            w = live ? tdw(s, p.s1, p.s2) : 0.f;         // second tile: w'
                            ds = w * (gvv - m_own);          // first tile: w' (gv - m)
                        } else {
                            const float2 stq = MODE == kModeDq ? st_own : s_b[(it & 1) * LT + blk * 32 + i];
                            ds = live ? fmaf(gvv, stq.x, stq.y) * tdw(s, p.s1, p.s2) : 0.f;
                            w *= stq.x;                      // dv_j = sum_i (w_ij / D_i) G_i
                        }
                        sr[i] = __float_as_uint(w);
                        gr[i] = __float_as_uint(ds);
                    }
                    uint32_t pw[16], pd[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        pw[i] = pack_bf16x2(__uint_as_float(sr[2 * i]), __uint_as_float(sr[2 * i + 1]));
                        pd[i] = pack_bf16x2(__uint_as_float(gr[2 * i]), __uint_as_float(gr[2 * i + 1]));
                    }
                    if (MODE == kModeDq) tmem_st16(tmem_addr(tb, lane_base, C::colD + blk * 16), pd);
                    if (MODE == kModeDqS) {
                        tmem_st16(tmem_addr(tb, lane_base, C::colD + blk * 16), pd);
                        tmem_st16(tmem_addr(tb, lane_base, C::colD2 + blk * 16), pw);
                    }
                    if (MODE == kModeFwd) tmem_st16(tmem_addr(tb, lane_base, C::colD + blk * 16), pw);
                    if (MODE == kModeDkDv) {
                        tmem_st16(tmem_addr(tb, lane_base, C::colS + blk * 16), pw);   // in place: columns already read
                        tmem_st16(tmem_addr(tb, lane_base, C::colG + blk * 16), pd);
                    }
                }
            };
            // uniform over the CTA: every pair of the tile is live
            const bool all_live = MODE == kModeDkDv ? (r0 + kTile - 1 <= c0 && c0 + LT <= p.L) : (c0 + LT - 1 <= r0);
            if (all_live) pass(std::false_type{});
            else pass(std::true_type{});
            if (MODE != kModeStats) tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&bars[bAlu]);
        }
        if (MODE != kModeStats) ok = rows_all(ok && mbar_wait(&bars[bFinal], 0, abort_flag));
        tc_fence_after();
        // tcgen05.ld is a warp-collective: every lane takes part, only the stores depend on the row
        const bool store = ok && row < p.L;
        const size_t grow = (size_t)head * p.L + (store ? row : 0);
        if (MODE == kModeStats || MODE == kModeDqS) {
            const float dinv = p.numerator_only ? 1.0f : 1.0f / (den + kEps);
            const float bq = p.numerator_only ? 0.0f : -en * dinv * dinv;
            if (store) p.stats_out[grow] = make_float2(dinv, bq);
            if (MODE == kModeDqS && ok) {
                // dq_i = X_i / D_i + (m_i / D_i + b_i) Y_i
                const float cy = fmaf(m_own, dinv, bq);
                uint32_t rx[16], ry[16];
                for (int h = 0; h < (p.df + 15) / 16; ++h) {     // p.df is uniform: 8, 16, 24, 32 gradient columns
                    tmem_ld16(tmem_addr(tb, lane_base, C::colAcc + h * 16), rx);
                    tmem_ld16(tmem_addr(tb, lane_base, C::colAcc2 + h * 16), ry);
                    tmem_wait_ld();
                    if (store) {
                        uint32_t o[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            o[i] = pack_bf16x2(fmaf(__uint_as_float(rx[2 * i]), dinv, cy * __uint_as_float(ry[2 * i])),
                                               fmaf(__uint_as_float(rx[2 * i + 1]), dinv, cy * __uint_as_float(ry[2 * i + 1])));
                        uint4* dst = reinterpret_cast<uint4*>(p.dq + grow * p.df + h * 16);
                        dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                        if (h * 16 + 8 < p.df) dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
                    }
                }
            }
        } else if (ok) {                                     // ok is uniform over the row threads (rows_all)
            // the d' gradient columns of dq (colAcc) or dk (colK), 16 at a time (p.df is uniform)
            for (int h = 0; h < (MODE == kModeFwd ? 0 : (p.df + 15) / 16); ++h) {
                uint32_t r[16];
                tmem_ld16(tmem_addr(tb, lane_base, (MODE == kModeDq ? C::colAcc : C::colK) + h * 16), r);
                tmem_wait_ld();
                if (store) {
                    uint4 o0, o1;
                    o0.x = pack_bf16x2(__uint_as_float(r[0]), __uint_as_float(r[1]));
                    o0.y = pack_bf16x2(__uint_as_float(r[2]), __uint_as_float(r[3]));
                    o0.z = pack_bf16x2(__uint_as_float(r[4]), __uint_as_float(r[5]));
                    o0.w = pack_bf16x2(__uint_as_float(r[6]), __uint_as_float(r[7]));
                    o1.x = pack_bf16x2(__uint_as_float(r[8]), __uint_as_float(r[9]));
                    o1.y = pack_bf16x2(__uint_as_float(r[10]), __uint_as_float(r[11]));
                    o1.z = pack_bf16x2(__uint_as_float(r[12]), __uint_as_float(r[13]));
                    o1.w = pack_bf16x2(__uint_as_float(r[14]), __uint_as_float(r[15]));
                    uint4* dst = reinterpret_cast<uint4*>((MODE == kModeDq ? p.dq : p.dk) + grow * p.df + h * 16);
                    dst[0] = o0;
                    if (h * 16 + 8 < p.df) dst[1] = o1;
                }
            }
            if (MODE == kModeDkDv || MODE == kModeFwd) {
                // the wide accumulator row: dv, or the forward output scaled by 1 / (denominator + eps)
                // through the own wide tile's place in shared memory (its products are done) in the layout of a TMA box,
                // [128 rows][64 columns] blocks with 128-byte rows, SWIZZLE_128B, and out by TMA: whole 128-byte lines
                // per row where a store per row thread would touch 32 rows per instruction.  Rows and columns past the
                // tensor's end are clipped by the store.
                const float sc = (MODE == kModeFwd && !p.numerator_only) ? 1.0f / (den + kEps) : 1.0f;
                for (int c = 0; c < p.dvw / 16; ++c) {       // p.dvw is uniform
                    uint32_t rv[16];
                    tmem_ld16(tmem_addr(tb, lane_base, C::colAcc + c * 16), rv);
                    tmem_wait_ld();
                    uint4 a, b;
                    a.x = pack_bf16x2(__uint_as_float(rv[0]) * sc, __uint_as_float(rv[1]) * sc);
                    a.y = pack_bf16x2(__uint_as_float(rv[2]) * sc, __uint_as_float(rv[3]) * sc);
                    a.z = pack_bf16x2(__uint_as_float(rv[4]) * sc, __uint_as_float(rv[5]) * sc);
                    a.w = pack_bf16x2(__uint_as_float(rv[6]) * sc, __uint_as_float(rv[7]) * sc);
                    b.x = pack_bf16x2(__uint_as_float(rv[8]) * sc, __uint_as_float(rv[9]) * sc);
                    b.y = pack_bf16x2(__uint_as_float(rv[10]) * sc, __uint_as_float(rv[11]) * sc);
                    b.z = pack_bf16x2(__uint_as_float(rv[12]) * sc, __uint_as_float(rv[13]) * sc);
                    b.w = pack_bf16x2(__uint_as_float(rv[14]) * sc, __uint_as_float(rv[15]) * sc);
                    uint8_t* rowp = smem + C::offResW + (c >> 2) * (kTile * 128) + t * 128;
                    *reinterpret_cast<uint4*>(rowp + ((((2 * c) & 7) ^ (t & 7)) << 4)) = a;
                    *reinterpret_cast<uint4*>(rowp + ((((2 * c + 1) & 7) ^ (t & 7)) << 4)) = b;
                }
                fence_proxy_async_smem();
                rows_all(true);
                if (t == 0) {
#pragma unroll
                    for (int bb = 0; bb < C::kVB; ++bb)
                        tma_store_3d(&tm_out, smem + C::offResW + bb * (kTile * 128), bb * 64, r0, head);
                    tma_store_commit();
                    tma_store_wait<0>();
                }
            }
        }
    }
    if (!ok && lane == 0) atomicOr(p.err, 1u);
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);     // loads still in flight get time to land
    }
    __syncthreads();
    if (warp == 4) tmem_dealloc(tb, C::kCols);
}

namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_fn_b() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}
// [BH][L][width] bf16, box = [1][128][box_w] (box_w may exceed width: the rest is zero-filled)
bool make_map_b(CUtensorMap* m, const void* base, int BH, int L, int width, int box_w, int box_rows,
                CUtensorMapSwizzle sw) {
    EncodeTiledFn enc = encode_fn_b();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)width, (cuuint64_t)L, (cuuint64_t)BH};
    cuuint64_t strides[2] = {(cuuint64_t)width * 2, (cuuint64_t)L * width * 2};
    cuuint32_t box[3] = {(cuuint32_t)box_w, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// the same map for the other tensor-core kernels of the library
bool make_rows_map_bf16(CUtensorMap* m, const void* base, int BH, int L, int width, int box_w, int box_rows,
                        CUtensorMapSwizzle sw) {
    return make_map_b(m, base, BH, L, width, box_w, box_rows, sw);
}

namespace {
// Block-wise path, between the passes.  state_scan_kernel: the per-block states of
// block_state_tc_kernel summed over the blocks before (suffix = 0) or after (suffix = 1) each
// block, as bf16 [BH x nblk][dvw][160] (tensor-core operand, transposed as the state kernel holds it) and fp32 row
// sums [BH x nblk][160].
__global__ void __launch_bounds__(256)
    state_scan_kernel(const float* __restrict__ part, const float* __restrict__ zpart, __nv_bfloat16* __restrict__ st,
                      float* __restrict__ sv, int nblk, int per, int suffix) {
    const int e = blockIdx.x * 256 + threadIdx.x;
    const size_t h0 = (size_t)blockIdx.y * nblk;
    if (e < per) {
        float run = 0.f;
        for (int i = 0; i < nblk; ++i) {
            const int c = suffix ? nblk - 1 - i : i;
            st[(h0 + c) * per + e] = __float2bfloat16(run);
            run += part[(h0 + c) * per + e];
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < 160) {
        float run = 0.f;
        for (int i = 0; i < nblk; ++i) {
            const int c = suffix ? nblk - 1 - i : i;
            sv[(h0 + c) * 160 + threadIdx.x] = run;
            run += zpart[(h0 + c) * 160 + threadIdx.x];
        }
    }
}
template <int DV, int MODE, int LT, bool XB = false>
based_status launch_pass(const CUtensorMap& n0, const CUtensorMap& w0, const CUtensorMap& n1, const CUtensorMap& w1,
                         const BParams& p, dim3 grid, const char* what, cudaStream_t stream,
                         const CUtensorMap* st = nullptr, const CUtensorMap* outm = nullptr) {
    using C = BCfg<DV, MODE, LT, XB>;
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BASED_ERR_CUDA;
    {
        std::lock_guard<std::mutex> lock(setup_mutex());
        if (!configured[dev]) {
            if (cudaFuncSetAttribute(backward_tc_kernel<DV, MODE, LT, XB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)C::kSmem) != cudaSuccess)
                return BASED_ERR_CUDA;
            configured[dev] = true;
        }
    }
    backward_tc_kernel<DV, MODE, LT, XB><<<grid, kThreadsB, C::kSmem, stream>>>(n0, w0, n1, w1, st ? *st : n0,
                                                                               outm ? *outm : w0, p);
    note_launch();
    return check_launch(what);
}

// Block length of the block-wise path, or 0 for the tile path alone.  The block-wise path needs d' = 16 and the
// statistics in one sweep (the forward output, or the numerator-only form); its cost grows with L where the tile
// path's grows with L^2, and the lengths below are where it starts to win on B200 (128 heads, d_v 64: 101 against
// 117 us at L = 768; d_v 128: 191 against 213 us at L = 1024; 32 heads, d_v 128: 129 against 134 us at L = 1536).
// Blocks of 256 tokens are the fastest from there on (B8 H16 L4096 d_v128: 613 / 582 / 661 us at 128 / 256 / 512),
// except with few heads at d_v 128, where every block's state costs a CTA of its own.
// A caller without the forward output gets it recomputed into the workspace first (one forward pass, 23 us at B4 H16
// L2048 d_v64, 83 us at B8 H16 L4096 d_v128), from somewhat longer sequences on.
int backward_block_len(int L, int df, bool merged, int d_v, int BH) {
    if (df != 16) return 0;
    if (!merged) {
        if (d_v == 64) return L >= 1024 ? 256 : 0;
        if (BH >= 64) return L >= 1536 ? 256 : 0;
        return L >= 4096 ? 512 : L >= 2048 ? 256 : 0;
    }
    if (d_v == 64) return L >= 768 ? 256 : 0;
    if (BH >= 64) return L >= 1024 ? 256 : 0;
    return L >= 4096 ? 512 : L >= 1536 ? 256 : 0;
}
size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
struct BlockWs {
    float* sv; float* zpart; float* part; __nv_bfloat16* st;
    __nv_bfloat16* out; void* fwd;                   // the recomputed forward output and the forward pass's own scratch
    size_t bytes;
};
// scratch after the [BH, L] float2 statistics
BlockWs block_ws(float* ws, int BH, int L, int dvr, int nblk) {
    BlockWs w{};
    const uintptr_t base = reinterpret_cast<uintptr_t>(ws);
    size_t off = align256((size_t)BH * L * 8);
    w.sv = reinterpret_cast<float*>(base + off);     off = align256(off + (size_t)BH * nblk * 160 * 4);
    w.zpart = reinterpret_cast<float*>(base + off);  off = align256(off + (size_t)BH * nblk * 160 * 4);
    // the blocks' own fp32 sums: only where a scan adds them up (few heads)
    w.part = reinterpret_cast<float*>(base + off);   off = align256(off + (BH >= 64 ? 0 : (size_t)BH * nblk * 160 * dvr * 4));
    w.st = reinterpret_cast<__nv_bfloat16*>(base + off);  off = align256(off + (size_t)BH * nblk * 160 * dvr * 2);
    w.out = reinterpret_cast<__nv_bfloat16*>(base + off); off = align256(off + (size_t)BH * L * dvr * 2);
    w.fwd = reinterpret_cast<void*>(base + off);     off = align256(off + prefill_tc_workspace_bytes(BH, L, dvr));
    w.bytes = off;
    return w;
}

template <int DV>
based_status launch_dvb(const void* q, const void* k, const void* v, const void* out, const void* g, void* dq, void* dk,
                        void* dv, float* ws, int BH, int L, int df, int dvr, int numerator_only, cudaStream_t stream) {
    constexpr int LTK = (DV == 64) ? 64 : 128;       // looped tile of the dk/dv pass (d_v 128 needs all 512 columns anyway)
    float2* stats = reinterpret_cast<float2*>(ws);
    // own tiles: 128 rows; looped tiles: 64 rows (and LTK rows for the dk/dv pass)
    CUtensorMap tq, tk, tv, tg, tk64, tv64, tqL, tgL, tdv;
    const CUtensorMapSwizzle s64 = CU_TENSOR_MAP_SWIZZLE_64B, s128 = CU_TENSOR_MAP_SWIZZLE_128B;
    if (!make_map_b(&tq, q, BH, L, df, 32, kTile, s64) || !make_map_b(&tk, k, BH, L, df, 32, kTile, s64) ||
        !make_map_b(&tv, v, BH, L, dvr, 64, kTile, s128) || !make_map_b(&tg, g, BH, L, dvr, 64, kTile, s128) ||
        !make_map_b(&tk64, k, BH, L, df, 32, 64, s64) || !make_map_b(&tv64, v, BH, L, dvr, 64, 64, s128) ||
        !make_map_b(&tqL, q, BH, L, df, 32, LTK, s64) || !make_map_b(&tgL, g, BH, L, dvr, 64, LTK, s128) ||
        !make_map_b(&tdv, dv, BH, L, dvr, 64, kTile, s128))
        return BASED_ERR_CUDA;
    BParams p{};
    if (error_word_ptr(&p.err) != BASED_OK) return BASED_ERR_CUDA;
    p.stats_in = stats;
    p.stats_out = stats;
    p.g_raw = static_cast<const __nv_bfloat16*>(g);
    p.o_raw = static_cast<const __nv_bfloat16*>(out);
    p.dq = static_cast<__nv_bfloat16*>(dq);
    p.dk = static_cast<__nv_bfloat16*>(dk);
    p.dvo = static_cast<__nv_bfloat16*>(dv);
    p.L = L;
    p.dvw = dvr;
    p.numerator_only = numerator_only;
    p.df = df;
    p.kdim = df <= 16 ? 16 : 32;
    p.s1 = 1.0f / sqrtf((float)df);
    p.s2 = 0.5f / (float)df;
    const dim3 grid((L + kTile - 1) / kTile, BH);
    based_status st;
    const int W = backward_block_len(L, df, out != nullptr || numerator_only, dvr, BH);
    if (W > 0) {
        // block-wise: pairs inside a block of W tokens by tiles, everything else through summed block states
        const int nblk = (L + W - 1) / W;
        const BlockWs w = block_ws(ws, BH, L, dvr, nblk);
        CUtensorMap tst;
        // the block states lie transposed, [BH x nblk][d_v][160]: boxes of 32 features x all value columns
        if (!make_map_b(&tst, w.st, BH * nblk, dvr, 160, 32, 64 * BCfg<DV, kModeDkDv, LTK>::kVB, s64)) return BASED_ERR_CUDA;
        if (out == nullptr && !numerator_only) {
            // the centre of the merged pass: the forward output, recomputed
            st = launch_prefill_tc(q, k, v, w.out, nullptr, nullptr, BH, L, dvr, 0, w.fwd, stream);
            if (st != BASED_OK) return st;
            p.o_raw = w.out;
        }
        p.W = W;
        p.nblk = nblk;
        p.sv = w.sv;
        // With many heads one CTA per head walks the blocks and writes the running sums; with few, one CTA per head
        // and block writes the block's own sums and a scan adds them up.
        const bool running = BH >= 64;
        auto states = [&](const void* x, const void* val, const void* sts, int rev) -> based_status {
            if (running) return launch_block_states_tc(x, val, sts, w.st, w.sv, nullptr, nullptr, BH, L, W, dvr, rev, stream);
            based_status s2 = launch_block_states_tc(x, val, sts, w.st, w.sv, w.part, w.zpart, BH, L, W, dvr, rev, stream);
            if (s2 != BASED_OK) return s2;
            state_scan_kernel<<<dim3((160 * dvr + 255) / 256, BH), 256, 0, stream>>>(w.part, w.zpart, w.st, w.sv, nblk, 160 * dvr, rev);
            note_launch();
            return check_launch("state_scan_kernel");
        };
        // states of the keys: S = sum mono(k) v^T, z = sum mono(k), summed over the blocks before each block
        if ((st = states(k, v, nullptr, 0)) != BASED_OK) return st;
        st = launch_pass<DV, kModeDqS, 64, true>(tq, tg, tk64, tv64, p, grid, "backward_tc_kernel<stats+dq, blocks>", stream, &tst);
        if (st != BASED_OK) return st;
        // states of the queries: R = sum mono(q) (dout / D)^T, R_b = sum b mono(q), summed over the blocks after each block
        if ((st = states(q, g, stats, 1)) != BASED_OK) return st;
        if (DV == 128) {
            // 32-row looped tiles: the accumulators then fit 256 tensor-memory columns and two CTAs share an SM, which
            // hides the fixed latency of these short-lived CTAs (273 -> 220 us for the pass at B8 H16 L4096)
            CUtensorMap tq32, tg32;
            if (!make_map_b(&tq32, q, BH, L, df, 32, 32, s64) || !make_map_b(&tg32, g, BH, L, dvr, 64, 32, s128)) return BASED_ERR_CUDA;
            return launch_pass<DV, kModeDkDv, 32, true>(tk, tv, tq32, tg32, p, grid, "backward_tc_kernel<dkdv, blocks>", stream, &tst,
                                                        &tdv);
        }
        return launch_pass<DV, kModeDkDv, LTK, true>(tk, tv, tqL, tgL, p, grid, "backward_tc_kernel<dkdv, blocks>", stream, &tst,
                                                     &tdv);
    }
    if (out != nullptr || numerator_only) {
        // statistics and dq in one sweep (needs the forward output as the centre of the packed products)
        st = launch_pass<DV, kModeDqS, 64>(tq, tg, tk64, tv64, p, grid, "backward_tc_kernel<stats+dq>", stream);
        if (st != BASED_OK) return st;
    } else {
        // statistics: own = queries (q, dout), looped = keys (k, v)
        st = launch_pass<DV, kModeStats, 64>(tq, tg, tk64, tv64, p, grid, "backward_tc_kernel<stats>", stream);
        if (st != BASED_OK) return st;
        // dq: own = queries (q, dout), looped = keys (k, v)
        st = launch_pass<DV, kModeDq, 64>(tq, tg, tk64, tv64, p, grid, "backward_tc_kernel<dq>", stream);
        if (st != BASED_OK) return st;
    }
    // dk, dv: own = keys (k, v), looped = queries (q, dout)
    return launch_pass<DV, kModeDkDv, LTK>(tk, tv, tqL, tgL, p, grid, "backward_tc_kernel<dkdv>", stream, nullptr, &tdv);
}
}  // namespace

// Forward of the definition form on the same tiles, for feature dimensions other than 16 (bf16 io,
// empty initial state): out = (sum_j w_ij v_j) / (sum_j w_ij + eps), w = 1 + s/sqrt(d') + s^2/(2 d').
based_status launch_quadratic_forward_tc(const void* q, const void* k, const void* v, void* out, int BH, int L,
                                         int d_feat, int d_v, int numerator_only, cudaStream_t stream) {
    CUtensorMap tq, tk64, tv64, tout;
    const CUtensorMapSwizzle s64 = CU_TENSOR_MAP_SWIZZLE_64B, s128 = CU_TENSOR_MAP_SWIZZLE_128B;
    if (!make_map_b(&tq, q, BH, L, d_feat, 32, kTile, s64) || !make_map_b(&tk64, k, BH, L, d_feat, 32, 64, s64) ||
        !make_map_b(&tv64, v, BH, L, d_v, 64, 64, s128) || !make_map_b(&tout, out, BH, L, d_v, 64, kTile, s128))
        return BASED_ERR_CUDA;
    BParams p{};
    if (error_word_ptr(&p.err) != BASED_OK) return BASED_ERR_CUDA;
    p.dvo = static_cast<__nv_bfloat16*>(out);
    p.L = L;
    p.dvw = d_v;
    p.numerator_only = numerator_only;
    p.df = d_feat;
    p.kdim = d_feat <= 16 ? 16 : 32;
    p.s1 = 1.0f / sqrtf((float)d_feat);
    p.s2 = 0.5f / (float)d_feat;
    const dim3 grid((L + kTile - 1) / kTile, BH);
    if (d_v == 64) return launch_pass<64, kModeFwd, 64>(tq, tq, tk64, tv64, p, grid, "quadratic forward (tc)", stream, nullptr, &tout);
    return launch_pass<128, kModeFwd, 64>(tq, tq, tk64, tv64, p, grid, "quadratic forward (tc)", stream, nullptr, &tout);
}

int backward_tc_block_tokens(int BH, int L, int d_feat, int d_v, int merged) {
    return backward_block_len(L, d_feat, merged != 0, d_v, BH);
}

size_t backward_tc_workspace_bytes(int BH, int L, int d_v) {
    const int W = backward_block_len(L, 16, true, d_v, BH);
    if (W > 0) return block_ws(nullptr, BH, L, d_v, (L + W - 1) / W).bytes;         // statistics, block states
    return (size_t)BH * L * 2 * sizeof(float);                 // (1 / D, b) per row
}

based_status launch_prefill_backward_tc(const void* q, const void* k, const void* v, const void* out, const void* g,
                                        void* dq, void* dk, void* dv, float* ws, int BH, int L, int d_feat, int d_v,
                                        int numerator_only, cudaStream_t stream) {
    if (d_v == 64) return launch_dvb<64>(q, k, v, out, g, dq, dk, dv, ws, BH, L, d_feat, 64, numerator_only, stream);
    return launch_dvb<128>(q, k, v, out, g, dq, dk, dv, ws, BH, L, d_feat, d_v, numerator_only, stream);  // 112 or 128
}

}  // namespace based

#ifdef BASED_TRACE
// debug builds: which barrier each warp of the first CTA that gave up was waiting on (this file's copy)
extern "C" void based_debug_read_waits_bwd(unsigned int* out) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(out, based::sm100::g_wait_dbg, sizeof(unsigned int) * 128);
    cudaMemcpyFromSymbol(out + 128, based::sm100::g_wait_owner, sizeof(unsigned int));
    unsigned int zero[129] = {};
    cudaMemcpyToSymbol(based::sm100::g_wait_dbg, zero, sizeof(unsigned int) * 128);
    cudaMemcpyToSymbol(based::sm100::g_wait_owner, zero, sizeof(unsigned int));
}
#endif
