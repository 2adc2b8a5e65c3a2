// Block states of the block-wise backward pass (bf16 io, d' = 16; Sec. 4.1, Eq. (3) applied to the
// gradients): running sums over a head's blocks of W tokens,
//
//   St[c][f][:] = s_f sum_t mono_f(x_t) u_t val_t      sv[c][f] = s_f sum_t mono_f(x_t) u_t wt_t
//
// over the tokens t of the blocks before block c (rev = 0: keys, x = k, val = v, u = 1, wt = 1) or
// after it (rev = 1: queries, x = q, val = dout, u_t = 1 / D_t, wt_t = b_t D_t, so that the row sum
// is sum_t b_t mono_f(q_t)).  mono_f are the 153 distinct monomials of the feature map, padded to
// 160 (f < 16: x_f | 16 + 16 o + m, o < 8: x_m x_(m+o) | 144 + m, m < 8: x_m x_(m+8) | 152: 1),
// s_f their weight in phi(q) . phi(k) (1/4 | 1/32 for o = 0, else 1/16 | 1/16 | 1).
//
// One CTA per head walks the 128-token tiles in order (rev: last to first), 288 threads: eight row
// warps, two threads per token of the step (and per accumulator lane at the block ends), each with
// half of the features; warp 8 issues TMA loads and MMAs (converged, one elected lane).  Per step the row threads form
// their token's 160 monomials times u_t in fp32, round once to bf16 and write them as a row of the B
// operand ([128 tokens][160], MN-major, five SWIZZLE_64B blocks of 32 features); the value tile comes
// by TMA and is the A operand as it lies ([128 tokens][d_v], MN-major), so the accumulator in tensor
// memory is the transposed state, [d_v lanes][160 columns] fp32.  The weights wt_t ride as two more
// rows of A (high and low bf16 part): lanes 64, 65 of the same accumulator at d_v 64, a second
// accumulator (M = 64) at d_v 112 / 128.  Two accumulators alternate from block to block: while the
// tensor pipe adds up the next block, the row threads read the finished one, add it to the running
// sums they keep in registers, scale, round to bf16 and write their lane's row of the next block's
// state, [d_v][160] - the layout the readers' descriptors take as it lies.  (The weights rows'
// accumulator at d_v 128 is never started over: blocks alternate between two pairs of its lanes,
// each pair a running sum of every second block.)  The operand tiles are double-buffered and the
// value tiles come through a ring of three stages.  With few heads one CTA per head and group of one
// to four consecutive blocks writes every block's own sums in fp32 instead, for a scan by another
// kernel.
#include <cuda_bf16.h>
#include <math.h>

#include <mutex>
#include <type_traits>

#include "common.cuh"
#include "sm100.cuh"

namespace based {
using namespace sm100;

bool make_rows_map_bf16(CUtensorMap* m, const void* base, int BH, int L, int width, int box_w, int box_rows,
                        CUtensorMapSwizzle sw);

namespace {
constexpr int kTok = 128;          // tokens per step
constexpr int kThreadsR = 288;     // eight row warps (two threads per token: half of its features each), one issuer warp
constexpr int kRowThreads = 256;
constexpr int kNSR = 3;            // value-tile stages
constexpr uint32_t kPhiBlk = kTok * 64;      // one block of 32 features: [128 tokens][64 bytes]
constexpr uint32_t kPhiBytes = 5 * kPhiBlk;

template <int DV> struct RCfg {
    static constexpr int kVB = (DV + 63) / 64;
    static constexpr uint32_t kVBytes = kVB * kTok * 128;      // [128 tokens][64 * kVB] bf16, SWIZZLE_128B blocks
    static constexpr uint32_t kWBytes = kTok * 128;            // weights block [128 tokens][64]: columns 0, 1
    static constexpr uint32_t offV = 0;
    static constexpr uint32_t offW = kNSR * kVBytes;
    static constexpr uint32_t offPhi = offW + 2 * kWBytes;
    static constexpr uint32_t offMisc = offPhi + 2 * kPhiBytes;
    static constexpr uint32_t kSmem = offMisc + 4096 + 1024;   // barriers; the row sums' parts (4 x 160 floats), their changes (2 x 160)
    // two accumulators of 160 columns that alternate from block to block; at d_v 128 the weights rows' accumulator
    static constexpr uint32_t colS = 0, colZ = 320;
    static constexpr uint32_t kCols = 512;
};
enum { rFull0 = 0, rAlu0 = 3, rMma0 = 5, rFlush0 = 7, rFree0 = 9, rNum = 11 };

struct RParams {
    const __nv_bfloat16* x;        // [BH, L, 16] k or q
    const float2* stats;           // (1 / D_t, b_t) per token, or null: u = 1, wt = 1
    __nv_bfloat16* st;             // [BH x nblk][160][dvw]
    float* sv;                     // [BH x nblk][160]
    // one CTA per (head, block) instead: the block's own sums in fp32, [BH x nblk][160][dvw] and [BH x nblk][160],
    // for a scan over the blocks by another kernel (few heads: the walk per head would leave most SMs idle)
    float* part;
    float* zpart;
    unsigned int* err;
    int L, dvw, W, nblk, rev;
    int grp;                       // own sums: blocks per CTA (consecutive blocks of one head)
};

// AND of a predicate over the 256 row threads (named barrier 3); also a barrier for their shared-memory traffic
__device__ __forceinline__ bool rows_and3(bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 3, 256, p;\n\t"
        "selp.b32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred)
        : "memory");
    return r != 0;
}
// one 256-bit store (the address a multiple of 32 bytes): a whole sector per lane where the lanes' rows lie apart
__device__ __forceinline__ void st_global_256(void* dst, const uint32_t (&w)[8]) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]),
                 "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                 : "memory");
}
__device__ __forceinline__ float feature_weight(int f) {
    return f < 16 ? 0.25f : f < 32 ? 0.03125f : f < 152 ? 0.0625f : f == 152 ? 1.0f : 0.0f;
}
}  // namespace

template <int DV>
__global__ void __launch_bounds__(kThreadsR, 1)
    block_state_tc_kernel(const __grid_constant__ CUtensorMap tm_val, const RParams p) {
    using C = RCfg<DV>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::offMisc);
    uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(bars + rNum);
    volatile uint32_t* abort_flag = tmem_base_s + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool own = p.part != nullptr;                      // every block's own sums, grp consecutive blocks per CTA
    const int ngrp = own ? (p.nblk + p.grp - 1) / p.grp : 1;
    const int head = own ? blockIdx.x / ngrp : blockIdx.x;
    const int blk = own ? (blockIdx.x % ngrp) * p.grp : 0;  // first block of the CTA
    const int spb = p.W / kTok;                              // steps per block
    const int ntile = (p.L + kTok - 1) / kTok;
    // running sums: the last block walked (first block in reverse) adds to no state that anyone reads
    const int nit = own ? min(p.grp * spb, ntile - blk * spb) : p.rev ? ntile - spb : (p.nblk - 1) * spb;
    auto tile_of = [&](int it) { return own ? blk * spb + it : p.rev ? ntile - 1 - it : it; };
    auto ends_block = [&](int it) {
        const int ti = tile_of(it);
        return own ? ((it + 1) % spb == 0 || it == nit - 1) : p.rev ? ti % spb == 0 : (ti + 1) % spb == 0;
    };

    if (tid == 0) {
        for (int s = 0; s < kNSR; ++s) mbar_init(&bars[rFull0 + s], 1);
        for (int b = 0; b < 2; ++b) { mbar_init(&bars[rAlu0 + b], kRowThreads); mbar_init(&bars[rMma0 + b], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&bars[rFlush0 + a], 1); mbar_init(&bars[rFree0 + a], kRowThreads); }
        *abort_flag = 0;
        fence_mbar_init();
    }
    for (int i = tid; i < 4 * 160; i += kThreadsR) reinterpret_cast<float*>(smem + C::offMisc + 256)[i] = 0.f;
    // the weights blocks: only the first eight bytes of a row are ever written again
    for (int i = tid; i < 2 * (int)C::kWBytes / 16; i += kThreadsR)
        reinterpret_cast<uint4*>(smem + C::offW)[i] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
    if (warp == 8) { tmem_alloc(tmem_base_s, C::kCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = *tmem_base_s;
    bool ok = true;

    if (warp == 8) {
        {
            // the whole warp runs this block; one elected lane issues the MMAs, commits and loads (see mma_ss_w)
            const uint32_t lead = elect_one();
            constexpr uint64_t dPhi = make_smem_desc_base(kPhiBlk, 512, kSwizzle64B);          // B, MN-major: 32-feature blocks
            constexpr uint64_t dV = make_smem_desc_base(kTok * 128, 1024, kSwizzle128B);       // A, MN-major: 64-column blocks
            constexpr uint32_t iS = make_idesc_bf16(128, 160, 1, 1);
            constexpr uint32_t iZ = make_idesc_bf16(64, 160, 1, 1);
            auto load = [&](int it) {
                if (!lead) return;
                const int s = it % kNSR;
                uint8_t* st = smem + C::offV + s * C::kVBytes;
                mbar_arrive_expect_tx(&bars[rFull0 + s], C::kVBytes);
#pragma unroll
                for (int b = 0; b < C::kVB; ++b)
                    tma_load_3d(st + b * (kTok * 128), &tm_val, &bars[rFull0 + s], b * 64, tile_of(it) * kTok, head);
            };
            for (int it = 0; it < kNSR && it < nit; ++it) load(it);
            int nblk_done = 0;                               // blocks walked so far: the accumulators alternate
            for (int it = 0; it < nit && ok; ++it) {
                const int b = it & 1, s = it % kNSR;
                const int a = nblk_done & 1;
                const bool first = it == 0 || ends_block(it - 1);        // first step of a block: the accumulator starts over
                ok = mbar_wait(&bars[rFull0 + s], (it / kNSR) & 1, abort_flag);
                if (!ok) break;
                ok = mbar_wait(&bars[rAlu0 + b], (it >> 1) & 1, abort_flag);
                if (!ok) break;
                // the row threads have read this accumulator's sums of two blocks ago
                if (first && nblk_done >= 2) {
                    ok = mbar_wait(&bars[rFree0 + a], ((nblk_done >> 1) - 1) & 1, abort_flag);
                    if (!ok) break;
                }
                tc_fence_after();
                const uint32_t dS = tb + C::colS + a * 160;
                const uint32_t aV = smem_u32(smem + C::offV + s * C::kVBytes);
                const uint32_t aW = smem_u32(smem + C::offW + b * C::kWBytes);
                const uint32_t lPhi = desc_lo(dPhi) + (smem_u32(smem + C::offPhi + b * kPhiBytes) >> 4);
                if (DV == 64) {
                    // rows 0..63 of A from the value tile, rows 64..127 from the weights block (its columns 0, 1)
                    const uint64_t dV1 = make_smem_desc_base(aW - aV, 1024, kSwizzle128B);
                    const uint32_t a_lo = desc_lo(dV1) + (aV >> 4), a_hi = desc_hi(dV1);
#pragma unroll
                    for (int k = 0; k < kTok / 16; ++k) {
                        if (first && k == 0)
                            mma_ss_w<false>(lead, dS, a_lo + k * 128, a_hi, lPhi + k * 64, desc_hi(dPhi), iS);
                        else
                            mma_ss_w<true>(lead, dS, a_lo + k * 128, a_hi, lPhi + k * 64, desc_hi(dPhi), iS);
                    }
                } else {
                    const uint32_t a_lo = desc_lo(dV) + (aV >> 4), w_lo = desc_lo(dV) + (aW >> 4);
#pragma unroll
                    for (int k = 0; k < kTok / 16; ++k) {
                        // the weights rows' accumulator is never started over: blocks alternate between two pairs of
                        // its lanes (the weights block's columns 0, 1 or 2, 3), each pair a running sum
                        if (first && k == 0) mma_ss_w<false>(lead, dS, a_lo + k * 128, desc_hi(dV), lPhi + k * 64, desc_hi(dPhi), iS);
                        else mma_ss_w<true>(lead, dS, a_lo + k * 128, desc_hi(dV), lPhi + k * 64, desc_hi(dPhi), iS);
                        if (it == 0 && k == 0)
                            mma_ss_w<false>(lead, tb + C::colZ, w_lo + k * 128, desc_hi(dV), lPhi + k * 64, desc_hi(dPhi), iZ);
                        else
                            mma_ss_w<true>(lead, tb + C::colZ, w_lo + k * 128, desc_hi(dV), lPhi + k * 64, desc_hi(dPhi), iZ);
                    }
                }
                mma_commit_w(lead, &bars[rMma0 + b]);
                if (ends_block(it)) {
                    mma_commit_w(lead, &bars[rFlush0 + a]);          // the block's sums are complete: the row threads read them
                    ++nblk_done;
                }
                // the previous step's products are done long since: its stage takes the load kNSR steps ahead
                if (it >= 1 && it - 1 + kNSR < nit) {
                    ok = mbar_wait(&bars[rMma0 + ((it - 1) & 1)], ((it - 1) >> 1) & 1, abort_flag);
                    if (!ok) break;
                    load(it - 1 + kNSR);
                }
            }
        }
    } else {
        // ===================================================================== row threads
        const int t = tid & 127;                             // token of the step; accumulator lane at the block ends
        const int half = tid >> 7;                           // features 0..79 or 80..159 of the token (columns of the lane)
        const uint32_t lane_base = (uint32_t)(warp & 3) * 32u;
        const uint32_t swz = (uint32_t)((t >> 1) & 3);
        // this step's row of x and its (1 / D, b), loaded one step ahead
        uint4 xa = make_uint4(0u, 0u, 0u, 0u), xb = xa;
        float2 sd = make_float2(0.f, 0.f);
        auto fetch = [&](int it) {
            const int tok = tile_of(it) * kTok + t;
            if (it < nit && tok < p.L) {
                const uint4* xp = reinterpret_cast<const uint4*>(p.x + ((size_t)head * p.L + tok) * 16);
                xa = xp[0];
                xb = xp[1];
                sd = p.stats ? p.stats[(size_t)head * p.L + tok] : make_float2(1.0f, 1.0f);
            } else {
                xa = make_uint4(0u, 0u, 0u, 0u);
                xb = xa;
                sd = make_float2(0.f, 0.f);                  // past the end: every monomial and the weight vanish
            }
        };
        // The sums over the blocks walked so far are the state of the next block in walking order: every lane's row
        // of the transposed state goes out as it lies, [slot][d_v][160] (bf16 running sums, or the block's own fp32
        // sums), the row sums through two small arrays in shared memory.
        float* zs = reinterpret_cast<float*>(smem + C::offMisc + 256);
        float* zd = zs + 4 * 160;
        float run[80];                                       // running sums of this thread's half of its lane's columns
#pragma unroll
        for (int i = 0; i < 80; ++i) run[i] = 0.f;
        auto flush = [&](int it, int nf) -> bool {
            const int a = nf & 1;
            if (!rows_and3(mbar_wait(&bars[rFlush0 + a], (nf >> 1) & 1, abort_flag))) return false;
            tc_fence_after();
            const int c = own ? blk + it / spb : p.rev ? tile_of(it) / spb - 1 : (tile_of(it) + 1) / spb;
            const size_t slot = (size_t)head * p.nblk + c;
            const size_t rowoff = (slot * p.dvw + (t < p.dvw ? t : 0)) * 160 + half * 80;
            // where the weights rows lie: d_v 64: lanes 64, 65 of this block's accumulator (own sums: added to the
            // running parts in shared memory); d_v 128: lanes 2a, 2a + 1 of their own accumulator (running sums of
            // every second block: they replace their parts, the other pair's parts stay as last read)
            const bool zwarp = (warp & 3) == (DV == 64 ? 2 : 0);
            const bool zlane = DV == 64 ? lane < 2 : (lane >> 1) == a;
            float* zrow = zs + lane * 160;                   // lanes 0..3 of the quarter: one part each
#pragma unroll
            for (int j = 0; j < 5; ++j) {
                uint32_t r[16];
                const int f0 = half * 80 + j * 16;           // this thread's half of the lane's columns
                tmem_ld16(tmem_addr(tb, lane_base, C::colS + a * 160 + f0), r);
                tmem_wait_ld();
                float v[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    run[j * 16 + i] += __uint_as_float(r[i]);
                    v[i] = run[j * 16 + i] * feature_weight(f0 + i);
                    if (own) run[j * 16 + i] = 0.f;              // own sums: every block starts over
                }
                if (t < p.dvw) {
                    if (own) {
                        uint32_t w8[8];
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) w8[i] = __float_as_uint(v[hh * 8 + i]);
                            st_global_256(p.part + rowoff + j * 16 + hh * 8, w8);
                        }
                    } else {
                        uint32_t o[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            __nv_bfloat162 h2 = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
                            o[i] = *reinterpret_cast<uint32_t*>(&h2);
                        }
                        st_global_256(p.st + rowoff + j * 16, o);       // 16 columns = one 32-byte sector of the lane's row
                    }
                }
                if (zwarp) {
                    if (DV != 64) {
                        tmem_ld16(tmem_addr(tb, lane_base, C::colZ + f0), r);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]) * feature_weight(f0 + i);
                    }
                    if (lane < 4 && zlane) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            // (d_v 128, own sums: the lane pair's running sum has grown by the block's own sum)
                            if (DV != 64 && own) zd[(lane & 1) * 160 + f0 + i] = v[i] - zrow[f0 + i];
                            zrow[f0 + i] = v[i];
                        }
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(&bars[rFree0 + a]);                  // the accumulator may start over
            const bool good = rows_and3(true);               // the row sums' parts are written
            if (tid < 160) {
                if (own && DV != 64) p.zpart[slot * 160 + tid] = zd[tid] + zd[160 + tid];
                else (own ? p.zpart : p.sv)[slot * 160 + tid] = (zs[tid] + zs[160 + tid]) + (zs[320 + tid] + zs[480 + tid]);
            }
            return rows_and3(good);                          // ... and read, before the next block end writes them
        };
        fetch(0);
        int nflush = 0, nflush_w = 0;                        // blocks read so far; blocks whose operands are written
        for (int it = 0; it < nit && ok; ++it) {
            const int b = it & 1;
            float x[16];
            {
                const __nv_bfloat162* ha = reinterpret_cast<const __nv_bfloat162*>(&xa);
                const __nv_bfloat162* hb = reinterpret_cast<const __nv_bfloat162*>(&xb);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 fa = __bfloat1622float2(ha[i]), fb = __bfloat1622float2(hb[i]);
                    x[2 * i] = fa.x; x[2 * i + 1] = fa.y;
                    x[8 + 2 * i] = fb.x; x[8 + 2 * i + 1] = fb.y;
                }
            }
            const float u = sd.x;
            // weight of the row sums: 1 for the keys; b_t D_t for the queries (the row itself carries 1 / D_t)
            const float wt = p.stats ? (u > 0.f ? sd.y / u : 0.f) : u;
            fetch(it + 1);
            // the operand buffers are free once the products of two steps ago are done
            ok = rows_and3(it < 2 || mbar_wait(&bars[rMma0 + b], ((it >> 1) - 1) & 1, abort_flag));
            if (!ok) break;
            uint8_t* prow = smem + C::offPhi + b * kPhiBytes + t * 64;
            float xu[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) xu[i] = x[i] * u;
            // ten 16-byte pieces (eight features each) per thread: pieces 0..9 or 10..19 of the row's twenty
            auto pieces = [&](auto half_tag) {
                constexpr int H = decltype(half_tag)::value;
#pragma unroll
                for (int q = 0; q < 10; ++q) {
                    const int g = H * 10 + q;                // piece of the row: block g / 4, position g % 4
                    uint32_t pk[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float mono[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int f = g * 8 + 2 * i + e;
                            const int m = f < 16 ? f : f < 144 ? ((f - 16) & 15) : f < 152 ? f - 144 : -1;
                            const int n = f < 16 ? -1 : f < 144 ? ((m + ((f - 16) >> 4)) & 15) : f < 152 ? m + 8 : -1;
                            mono[e] = f > 152 ? 0.f : m < 0 ? u : n < 0 ? xu[m] : xu[m] * x[n];
                        }
                        __nv_bfloat162 h2 = __floats2bfloat162_rn(mono[0], mono[1]);
                        pk[i] = *reinterpret_cast<uint32_t*>(&h2);
                    }
                    *reinterpret_cast<uint4*>(prow + (g >> 2) * kPhiBlk + (((g & 3) ^ swz) << 4)) =
                        make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
            };
            if (half == 0) pieces(std::integral_constant<int, 0>{});
            else pieces(std::integral_constant<int, 1>{});
            if (half == 0) {
                // the token's weight, high and low part, as two columns of its row of the weights block: 0 and 1, or
                // at d_v 128 2 and 3 in every second block (the other pair zero)
                __nv_bfloat16 hi = __float2bfloat16(wt), lo = __float2bfloat16(wt - __bfloat162float(hi));
                __nv_bfloat162 h2;
                h2.x = hi;
                h2.y = lo;
                const uint32_t w2 = *reinterpret_cast<uint32_t*>(&h2);
                const bool second = DV != 64 && (nflush_w & 1);
                *reinterpret_cast<uint2*>(smem + C::offW + b * C::kWBytes + t * 128 + ((t & 7) << 4)) =
                    second ? make_uint2(0u, w2) : make_uint2(w2, 0u);
            }
            if (ends_block(it)) ++nflush_w;
            fence_proxy_async_smem();
            mbar_arrive(&bars[rAlu0 + b]);
            // a block ended with the step before: its sums are read after this step's operand is handed over, so
            // that the tensor pipe has work the moment the read is done
            if (it > 0 && ends_block(it - 1)) {
                ok = flush(it - 1, nflush++);
                if (!ok) break;
            }
        }
        if (ok && nit > 0 && ends_block(nit - 1)) ok = flush(nit - 1, nflush++);
    }
    if (!ok && lane == 0) atomicOr(p.err, 1u);
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);     // loads still in flight get time to land
    }
    __syncthreads();
    if (warp == 8) tmem_dealloc(tb, C::kCols);
}

namespace {
template <int DV>
based_status launch_running(const void* x, const void* val, const float2* stats, void* st, float* sv, float* part,
                            float* zpart, int BH, int L, int W, int dvw, int rev, cudaStream_t stream) {
    using C = RCfg<DV>;
    CUtensorMap tv;
    if (!make_rows_map_bf16(&tv, val, BH, L, dvw, 64, kTok, CU_TENSOR_MAP_SWIZZLE_128B)) return BASED_ERR_CUDA;
    RParams p{};
    if (error_word_ptr(&p.err) != BASED_OK) return BASED_ERR_CUDA;
    p.x = static_cast<const __nv_bfloat16*>(x);
    p.stats = stats;
    p.st = static_cast<__nv_bfloat16*>(st);
    p.sv = sv;
    p.part = part;
    p.zpart = zpart;
    p.L = L;
    p.dvw = dvw;
    p.W = W;
    p.nblk = (L + W - 1) / W;
    p.rev = rev;
    // own sums: enough consecutive blocks per CTA to spread its fixed cost, while some waves of CTAs remain
    // (B1 H32 L32768 d_v64: 1170 / 1099 / 1061 / 1078 us per backward call at 1 / 2 / 4 / 8 blocks per CTA)
    p.grp = !part ? 1 : BH * p.nblk >= 1200 ? 4 : BH * p.nblk >= 600 ? 2 : 1;
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BASED_ERR_CUDA;
    {
        std::lock_guard<std::mutex> lock(setup_mutex());
        if (!configured[dev]) {
            if (cudaFuncSetAttribute(block_state_tc_kernel<DV>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)C::kSmem) != cudaSuccess)
                return BASED_ERR_CUDA;
            configured[dev] = true;
        }
    }
    block_state_tc_kernel<DV><<<part ? BH * ((p.nblk + p.grp - 1) / p.grp) : BH, kThreadsR, C::kSmem, stream>>>(tv, p);
    note_launch();
    return check_launch("block_state_tc_kernel");
}
}  // namespace

// W: a multiple of 128, L > W.  stats: (1 / D_t, b_t) per token for the query side, null for the key side.
// part, zpart: null for the running sums (one CTA per head); else every block's own sums go there in fp32 (one CTA
// per head and block) and st, sv stay untouched.
based_status launch_block_states_tc(const void* x, const void* val, const void* stats, void* st, float* sv, float* part,
                                    float* zpart, int BH, int L, int W, int d_v, int rev, cudaStream_t stream) {
    const float2* s2 = static_cast<const float2*>(stats);
    if (d_v == 64) return launch_running<64>(x, val, s2, st, sv, part, zpart, BH, L, W, 64, rev, stream);
    return launch_running<128>(x, val, s2, st, sv, part, zpart, BH, L, W, d_v, rev, stream);        // 112 or 128
}

}  // namespace based
