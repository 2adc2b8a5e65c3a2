// based_prefill, bf16 tensor-core path (tcgen05 + TMEM + TMA, sm_100a).
//
// Causal Taylor linear attention (Sec. 4.1, Eq. (2)/(3)) evaluated chunk by chunk as in
// Sec. 5.2: within a chunk of 128 tokens the quadratic "attention" form, across chunks
// the running KV-state.  Unlike Algorithm 1 the whole expanded state of a head lives in
// tensor memory as one fp32 accumulator, and the expanded features never leave the SM.
//
// Per chunk c of one (b, h) (or of one sequence segment of it) the tensor-core steps are
//   (1) scores   T[128,128]  = Q_c K_c^T                        (K = 16)
//   (5) S^T     += V_c^T phi(K_c)           [d_v lanes x 160 feature columns, fp32 in TMEM]
//   (z) z       += colsum(phi(K_c))         d_v = 64: an extra "ones" column of V, i.e. lane 64
//                                           of S^T; d_v = 128: phi(K_c)^T x ones (N = 16)
//   (4) Y        = phi(Q_c) [S_prev | z_prev]   (K = 160; the extra column is the
//                                                cross-chunk part of the denominator)
//   (3) Y       += P V_c,  P = (1 + T/4 + T^2/32) masked to j <= i, bf16, read from TMEM
// and the ALU jobs: polynomial + mask + row sum on the scores, expansion of q and k rows
// into feature rows (shared memory, UMMA operand layout), a bf16 copy of the fp32 state
// as the B operand of (4), and normalise + store through shared memory and TMA.
//
// Features are kept in a symmetric basis of 153 (padded to 160) instead of 273: with
// x' = x/2,  [x' (16) | x'_m x'_(m+o) for o = 0..7 (the o = 0 block scaled by 1/sqrt 2) |
// x'_m x'_(m+8), m < 8 | 1 | 0 x 7].  Its inner products equal those of the 273-feature
// map; the state is expanded to / folded from the 273-row ABI layout at the kernel's edges.
//
// Warp roles (608 threads): warps 0-3 "row" group (one thread per query row: polynomial),
// warps 4-7 "feature" group (one thread per token: phi expansion), warps 8-11 "state"
// group (one thread per TMEM lane: bf16 state copy, state I/O), warps 12-15 "output"
// group (one thread per output row: normalise, stage, TMA store), warp 16 TMA producer,
// warp 17 issues the state-update MMAs (5)/(z), warp 18 the output-side MMAs (1)/(4)/(3):
// two independent in-order streams, so the state chain runs ahead of the output chain; both
// warps run converged and predicate only the MMA and its commit on one elected lane (sm100.cuh).
// All cross-role hand-offs are mbarriers with bounded waits.  A piece that ends its head (or, in
// the state pass, its range) has its final state written by all four groups, a quarter each.
//
// d_v 64, plain chunk loop: phi(Q) does not go through shared memory.  The feature group writes it
// into tensor memory (the upper half of the chunk's score buffer once the row group has read the
// scores, plus 16 spare columns) as the A operand of step (4), and the shared-memory tile that
// frees holds a second state-copy tile, so the copy for chunk c+1 is written while step (4) of
// chunk c reads its own.
// d_v 128, plain chunk loop: features 0..95 of phi(Q) go to the 48 tensor-memory columns behind
// the z tiles, features 96..159 to shared memory; the rest of the phi(Q) tile's place is a second
// output staging tile, and the output group releases the accumulator before it stages anything.
#include <cuda_bf16.h>
#include <cstdlib>

#include "common.cuh"
#include "sm100.cuh"

namespace based {

using namespace sm100;

namespace {

constexpr int kC = 128;            // tokens per chunk
constexpr int kF = 160;            // internal feature count (153 padded to a multiple of 16)
constexpr int kFBlk = 5;           // 32-feature SWIZZLE_64B blocks
constexpr int kThreads = 608;
constexpr int kModeMain = 0, kModeState = 1, kModePre = 2;
constexpr int kWarpTma = 16, kWarpMma = 17, kWarpMmaY = 18;
constexpr float kRsqrt2 = 0.70710678118654752f;

// ---- workspace layout of one (head, segment) partial state: [kF][DV] fp32 then [kF] fp32
__host__ __device__ constexpr size_t seg_state_floats(int dv) { return (size_t)kF * dv + kF; }

template <int DV>
struct Cfg {
    // d_v 64: four stages (a tile's load takes about 2500 cycles from issue to arrival, more than a chunk's period;
    // with three the next chunk's scores waited for their tile: measured 5-8 % on the 360M shapes)
    static constexpr int kStages = (DV == 64) ? 4 : 2;
    // The state pass loads no q tile and needs neither state copy nor output staging, and what bounds it is the bytes
    // in flight (20 KB per stage and SM, about 2500 cycles per load: four stages are 4.7 TB/s over 148 SMs), so its
    // stages are packed (k tile, v tile) and there are as many as fit in front of the ones block and two phi(K) tiles
    static constexpr int kStagesState = (DV == 64) ? 6 : 3;
    // How a piece of the main pass gets the state of the pieces before it in its head (up to seven workspace slots,
    // or one per earlier range, of 40-80 KB each).  Its state group reading them alone spends 2.7 us of load latency
    // per slot before the first state update can run (11 us on cfg 5's last pieces, 46 us with 18 pieces per head).
    // d_v 128: all four role groups share the read (init_state_blocks).  d_v 64: a small kernel between the two
    // passes turns the slots into running sums (slot_scan_kernel) and the piece reads one slot; sharing the read
    // as at d_v 128 was as fast there, but every form of it tried slowed that kernel's role loops by 3-18 %
    // (register allocation), on shapes that have no slots at all.
    static constexpr bool kSlotScan = DV == 64;
    static constexpr int kNY = DV + 16;                         // Y columns: d_v numerators + denominator block
    static constexpr int kSLanes = (DV == 64) ? 65 : 128;       // live lanes of S^T (d_v 64: lane 64 carries z)
    static constexpr uint32_t kQKBytes = kC * 32;               // one q or k tile (16 bf16 per token)
    static constexpr uint32_t kVBytes = kC * DV * 2;
    static constexpr uint32_t kStageBytes = 2 * kQKBytes + kVBytes;
    static constexpr uint32_t kPhiBlk = kC * 64;                // bytes of one 32-feature block
    static constexpr uint32_t kPhiBytes = kFBlk * kPhiBlk;      // 40 KB
    static constexpr uint32_t kScBlk = kNY * 64;
    static constexpr uint32_t kScBytes = kFBlk * kScBlk;
    // d_v 64: a [16 tokens][64] bf16 block whose column 0 is 1.0: the second 64-wide block of V^T (and of V) for one
    // K-step of 16 tokens.  Every K-step's block would hold the same, so all of them read this one: the descriptor
    // of K-step k starts 2 KB further and its block offset is 2 KB shorter.
    // d_v 128: a block of bf16 ones (B operand of the z step)
    static constexpr uint32_t kOnesBytes = 2048;
    static constexpr uint32_t kOutBytes = kC * 128;             // staging of 64 output columns
    static constexpr uint32_t offStage = 0;
    static constexpr uint32_t offOnes = kStages * kStageBytes;  // after the stages: LBO of V^T stays positive
    static constexpr uint32_t offPK = offOnes + kOnesBytes;
    static constexpr uint32_t offPQ = offPK + kPhiBytes;        // must follow PK (the last z tile over-reads into it)
    static constexpr uint32_t offSc = offPQ + kPhiBytes;
    static constexpr uint32_t offOut = offSc + kScBytes;
    static constexpr uint32_t offMisc = offOut + kOutBytes;
    static constexpr uint32_t kMiscBytes = 3072;                // barriers, row sums, ABI row table, the CTA's piece
    static constexpr uint32_t kSmemBytes = offMisc + kMiscBytes + 1024;   // + alignment slack
    static_assert(kSmemBytes <= 232448, "shared memory budget");
    // TMEM columns
    static constexpr uint32_t colT = 0;                          // scores, overwritten in place by P
    static constexpr bool kTDouble = (DV == 64);                 // two score buffers when TMEM has room
    static constexpr uint32_t colY = kTDouble ? 256 : 128;
    static constexpr uint32_t colS = colY + kNY;
    static constexpr uint32_t colZ0 = colS + kF;                 // d_v 128 only
    static constexpr uint32_t colZ1 = colZ0 + 16;
    // d_v 64: phi(Q) of a chunk lives in tensor memory as the A operand of step (4): features 0..127 in
    // the upper half of the chunk's score buffer (free once the row group has read the scores), features
    // 128..159 in the 16 columns after the state; the shared-memory tile it leaves free during the own
    // chunks holds a second copy tile of the state, so the state group writes chunk c+1's copy while
    // step (4) of chunk c still reads its own
    static constexpr bool kPQinT = (DV == 64);
    static constexpr uint32_t colPQhi = colS + kF;
    static_assert((DV == 64 ? colS + kF + 16 : colZ1 + 16) <= 512, "TMEM budget");
    // d_v 128, plain chunk loop: the 48 columns behind the z tiles hold features 0..95 of phi(Q) (A operand of the
    // first six K-steps of step (4)); only features 96..159 stay in shared memory, two blocks at the start of the
    // phi(Q) tile's place, and the 16 KB behind them are a second output staging tile
    static constexpr uint32_t colPQlo = colZ1 + 16;
    static constexpr uint32_t offOut2 = offPQ + 2 * kPhiBlk;
    static_assert(kScBlk % 1024 == 0 && kStageBytes % 1024 == 0 && offPK % 1024 == 0, "tiles stay 1024-byte aligned");
};

enum Bar {
    kFull0 = 0, kEmpty0 = 8, kG1 = 16, kG1b, kP, kPb, kG2, kG2b, kG4, kG4b, kG3, kR4, kPK, kPKb, kSR, kDone, kTR, kTRb, kSC, kSCb, kFin, kInit,
    kNumBars
};

// segments per head, chunks per segment (the last one takes the rest), mode
struct SegPlan { int nseg; int per; bool recompute; int balanced; };   // balanced > 0: that many equal chunk ranges over all heads

struct Params {
    float* kv_abi;        // [BH, 273, DV] or null
    float* z_abi;         // [BH, 273] or null
    float* ws;            // per (head, segment) partial states, internal layout
    unsigned int* err;
    int L;                // tokens per head
    int nseg;             // segments per head
    int seg_len;          // tokens per segment (multiple of kC)
    int continue_abi;     // start from the ABI state in kv_abi / z_abi
    int sym;              // kv_abi / z_abi use the 153-row symmetric format
    int numerator_only;   // outputs are not divided by the denominator
    int dv;               // value head dimension of the caller's tensors (112 runs on the d_v 128 kernel:
                          // the tensor maps zero-fill columns 112..127 on load and clip them on store)
    int balanced;         // > 0: the number of equal chunk ranges the heads' chunks are cut into (see the kernel)
    int heads;            // B*H (balanced mode)
    int pad;              // balanced mode: chunks counted in front of every head for the CTA it starts;
                          // segments with a state pass: 1 if each head's first slot holds the caller's state
#ifdef BASED_TRACE
    unsigned long long* trace;
#endif
};

#if defined(BASED_TRACE) && !defined(BASED_TRACE_CTA_ONLY)
#define TRACE(role, c, ev)                                                                   \
    do {                                                                                     \
        if (p.trace && blockIdx.x == gridDim.x - 1 && blockIdx.y == 0 && (c) >= 0 && (c) < 64)           \
            p.trace[((role) * 64 + (c)) * 8 + (ev)] = clock64();                             \
    } while (0)
#else
#define TRACE(role, c, ev) do {} while (0)
#endif
#ifdef BASED_TRACE
// wall-clock entry / exit of every CTA (with its SM), after the per-role events (state pass: 2048 entries further on)
#define TRACE_CTA(which)                                                                                      \
    do {                                                                                                      \
        if (p.trace) p.trace[6 * 64 * 8 + ((MODE == kModeState ? 2048 : 0) + blockIdx.y * gridDim.x + blockIdx.x) * 2 + (which)] = (global_timer_ns() << 8) | smid_u32(); \
    } while (0)
#else
#define TRACE_CTA(which) do {} while (0)
#endif

// ---- internal feature index -> rows of the 273-row ABI layout -------------------------
struct AbiRows { int a, b; };   // b < 0: single row (scale 1); b >= 0: two rows, scale 1/sqrt 2; a < 0: padding
__host__ __device__ constexpr AbiRows abi_rows(int i) {
    if (i < 16) return {1 + i, -1};
    if (i < 144) {
        const int o = (i - 16) / 16, m = (i - 16) % 16, n = (m + o) % 16;
        if (o == 0) return {17 + 17 * m, -1};
        return {17 + 16 * m + n, 17 + 16 * n + m};
    }
    if (i < 152) {
        const int m = i - 144, n = m + 8;
        return {17 + 16 * m + n, 17 + 16 * n + m};
    }
    if (i == 152) return {0, -1};
    return {-1, -1};
}

// ---- the same for the 153-row symmetric state format: the internal basis is that format's
// feature set in another order, so every feature maps to one row with scale 1
__host__ __device__ constexpr AbiRows sym_rows(int i) {
    if (i < 16) return {1 + i, -1};
    if (i < 144) {
        const int o = (i - 16) / 16, m = (i - 16) % 16, n = (m + o) % 16;
        return {m <= n ? sym_pair_row(m, n) : sym_pair_row(n, m), -1};
    }
    if (i < 152) return {sym_pair_row(i - 144, i - 144 + 8), -1};
    if (i == 152) return {0, -1};
    return {-1, -1};
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t mul2(uint32_t a, uint32_t b) {
    __nv_bfloat162 r = __hmul2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
    return *reinterpret_cast<uint32_t*>(&r);
}

// Expand one raw 16-vector (8 packed bf16 pairs) into its 160 internal features: 20 packed
// 16-byte pieces f[0..19] (piece j = features 8j .. 8j+7).
__device__ __forceinline__ void compute_phi_row(uint4 xlo, uint4 xhi, bool valid, uint4 (&f)[20]) {
    const uint32_t x[8] = {xlo.x, xlo.y, xlo.z, xlo.w, xhi.x, xhi.y, xhi.z, xhi.w};
    const uint32_t kHalf = 0x3F003F00u;      // (0.5, 0.5)
    const uint32_t kRs2 = 0x3F353F35u;       // (1/sqrt2, 1/sqrt2) rounded to bf16
    uint32_t E[8], O[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) E[i] = valid ? mul2(x[i], kHalf) : 0u;
#pragma unroll
    for (int i = 0; i < 8; ++i) O[i] = __byte_perm(E[i], E[(i + 1) & 7], 0x5432);   // (x'_{2i+1}, x'_{2i+2})
    f[0] = make_uint4(E[0], E[1], E[2], E[3]);
    f[1] = make_uint4(E[4], E[5], E[6], E[7]);
    {   // o = 0: squares, scaled by 1/sqrt 2
        uint32_t p[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) p[i] = mul2(E[i], mul2(E[i], kRs2));
        f[2] = make_uint4(p[0], p[1], p[2], p[3]);
        f[3] = make_uint4(p[4], p[5], p[6], p[7]);
    }
#pragma unroll
    for (int o = 1; o < 8; ++o) {
        uint32_t p[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t r = (o & 1) ? O[(i + (o - 1) / 2) & 7] : E[(i + o / 2) & 7];
            p[i] = mul2(E[i], r);
        }
        f[2 + 2 * o] = make_uint4(p[0], p[1], p[2], p[3]);
        f[3 + 2 * o] = make_uint4(p[4], p[5], p[6], p[7]);
    }
    f[18] = make_uint4(mul2(E[0], E[4]), mul2(E[1], E[5]), mul2(E[2], E[6]), mul2(E[3], E[7]));
    f[19] = make_uint4(valid ? 0x00003F80u : 0u, 0u, 0u, 0u);   // the constant feature 1.0
}

// The same expansion one 32-feature block (16 packed registers) at a time, for callers that store each block as it
// is formed: block 0 = x' and the squares, block j = the products of offsets 2j-1 and 2j, block 4 = offset 7, the
// eight products of offset 8, the constant.  E and O as in compute_phi_row.
__device__ __forceinline__ void phi_prepare(uint4 xlo, uint4 xhi, bool valid, uint32_t (&E)[8], uint32_t (&O)[8]) {
    const uint32_t x[8] = {xlo.x, xlo.y, xlo.z, xlo.w, xhi.x, xhi.y, xhi.z, xhi.w};
    const uint32_t kHalf = 0x3F003F00u;
#pragma unroll
    for (int i = 0; i < 8; ++i) E[i] = valid ? mul2(x[i], kHalf) : 0u;
#pragma unroll
    for (int i = 0; i < 8; ++i) O[i] = __byte_perm(E[i], E[(i + 1) & 7], 0x5432);
}
template <int J>
__device__ __forceinline__ void phi_block(const uint32_t (&E)[8], const uint32_t (&O)[8], bool valid, uint32_t (&v)[16]) {
    const uint32_t kRs2 = 0x3F353F35u;
    if constexpr (J == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) { v[i] = E[i]; v[8 + i] = mul2(E[i], mul2(E[i], kRs2)); }
    } else if constexpr (J < 4) {
#pragma unroll
        for (int i = 0; i < 8; ++i) { v[i] = mul2(E[i], O[(i + J - 1) & 7]); v[8 + i] = mul2(E[i], E[(i + J) & 7]); }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = mul2(E[i], O[(i + 3) & 7]);
#pragma unroll
        for (int i = 0; i < 4; ++i) v[8 + i] = mul2(E[i], E[i + 4]);
        v[12] = valid ? 0x00003F80u : 0u;
        v[13] = v[14] = v[15] = 0u;
    }
}

// Write the 20 pieces as row t of a [128 tokens][160 features] tile made of five SWIZZLE_64B blocks.
__device__ __forceinline__ void store_phi_row(const uint4 (&f)[20], uint8_t* tile, int t) {
    uint8_t* row = tile + (t >> 3) * 512 + (t & 7) * 64;
    const uint32_t sw = (t >> 1) & 3;
#pragma unroll
    for (int j = 0; j < 20; ++j)
        *reinterpret_cast<uint4*>(row + (j >> 2) * (kC * 64) + (((j & 3) ^ sw) << 4)) = f[j];
}

__device__ __noinline__ void write_phi_row(uint4 xlo, uint4 xhi, uint8_t* tile, int t, bool valid) {
    uint4 f[20];
    compute_phi_row(xlo, xhi, valid, f);
    store_phi_row(f, tile, t);
}

// Row t of a [128][16] bf16 tile written by TMA with SWIZZLE_32B.
__device__ __forceinline__ void read_qk_row(const uint8_t* tile, int t, uint4& lo, uint4& hi) {
    const uint8_t* row = tile + (t >> 3) * 256 + (t & 7) * 32;
    const uint32_t sw = ((t >> 2) & 1) << 4;
    lo = *reinterpret_cast<const uint4*>(row + (0 ^ sw));
    hi = *reinterpret_cast<const uint4*>(row + (16 ^ sw));
}

// Packed fp32 pairs (sm_100 has two-wide fp32 multiply-add and add): a pair lives in one 64-bit register.
__device__ __forceinline__ uint64_t f32x2(uint32_t lo, uint32_t hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void f32x2_split(uint64_t v, float& lo, float& hi) {
    uint32_t a, b;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
    lo = __uint_as_float(a);
    hi = __uint_as_float(b);
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t mul2f(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
// two fp32 accumulator columns scaled and packed to bf16: one two-wide multiply and one conversion
__device__ __forceinline__ uint32_t scale_pack(uint32_t y0, uint32_t y1, uint64_t inv2) {
    float lo, hi;
    f32x2_split(mul2f(f32x2(y0, y1), inv2), lo, hi);
    return pack_bf16(lo, hi);
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ void group_sync(int id) {        // named barrier of one 128-thread group
    asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory");
}
// AND of a predicate over one 128-thread group (every thread gets the same answer, so the
// group leaves its loop together and never strands a member at a named barrier)
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

}  // namespace

// MODE: kModeMain = chunk loop from a given initial state; kModeState = state-update-only pass over
// a segment (partial state to the workspace); kModePre = kModeMain preceded by state-update-only
// "pre-chunks" over everything before the segment (recompute mode).
// ---- initial state.  One thread per TMEM lane of the state accumulator S^T; lane t of a warp's lane quarter holds
// V column t (d_v 64: lane 64 the K-state).  Its initial value is the caller's ABI state (folded into the internal
// basis; kv_abi == nullptr: none) plus the partial states of the earlier pieces (nprev workspace slots from wsh on).
// Those are up to seven slots of 40-80 KB each, read as ten 16-column blocks per slot, and one thread group doing it
// alone spends 0.7 us of load latency per block and slot before the first state update can run (2.7 us per slot).
// So in the main pass all four role groups (each has a warp per lane quarter) take every fourth block (part of
// nparts), and two slots' loads are in flight at a time; the state group waits for the others before it reads the
// state.  Not inlined: its registers are its own and the role loops' allocation does not see it.
template <int DV>
__device__ __noinline__ void init_state_blocks(const float* wsh, int nprev, bool wait_for_state_pass, const float* kv_abi,
                                               const float* z_abi, int dv, int abi_row0, const short2* s_abi, uint32_t tb,
                                               int part, int nparts) {
    using C = Cfg<DV>;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t lane_base = (uint32_t)(warp & 3) * 32u;
    const int t = ((warp & 3) << 5) + lane;
    // what this thread's lane of S^T holds: V column srow, or (d_v 64) the K-state at lane 64
    const int srow = (t < C::kSLanes) ? t : -1;
    const bool is_z = (DV == 64) && t == 64;
    // d_v 128: K-state features held in the two z tiles (64-row MMA: rows 0..31 in lanes 0-15, 32-47)
    const int z1f = (DV == 128 && (t & 31) < 16 && (t >> 5) < 2) ? 128 + (t >> 5) * 16 + (t & 15) : -1;
    const size_t seg_stride = seg_state_floats(DV);
    const bool from_abi = kv_abi != nullptr;            // dv: row pitch of the caller's state; lanes >= dv hold zeros
    const float* kvh = from_abi ? kv_abi + (size_t)abi_row0 * dv : nullptr;
    const float* zh = from_abi ? z_abi + abi_row0 : nullptr;
    // the partial states are the state pass's output (a no-op when this grid was launched the plain way)
    if (wait_for_state_pass) asm volatile("griddepcontrol.wait;" ::: "memory");
#pragma unroll 1
    for (int b = part; b < kF / 16; b += nparts) {
        float acc[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) acc[i] = 0.f;
        if (srow >= 0) {
            if (from_abi) {
                float va[16], vb[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const short2 ar = s_abi[b * 16 + i];
                    const bool live = is_z || srow < dv;
                    va[i] = (ar.x >= 0 && live) ? (is_z ? zh[ar.x] : kvh[(size_t)ar.x * dv + srow]) : 0.f;
                    vb[i] = (ar.y >= 0 && live) ? (is_z ? zh[ar.y] : kvh[(size_t)ar.y * dv + srow]) : 0.f;
                }
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[i] = (s_abi[b * 16 + i].y >= 0) ? (va[i] + vb[i]) * kRsqrt2 : va[i];
            }
            const float* src = wsh + (is_z ? (size_t)kF * DV + b * 16 : (size_t)(b * 16) * DV + srow);
            const size_t step = is_z ? 1 : DV;
            int sp = 0;
#pragma unroll 1
            for (; sp + 1 < nprev; sp += 2, src += 2 * seg_stride) {
                float t0[16], t1[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) { t0[i] = src[i * step]; t1[i] = src[seg_stride + i * step]; }
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[i] += t0[i] + t1[i];
            }
            if (sp < nprev) {
                float t0[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) t0[i] = src[i * step];
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[i] += t0[i];
            }
        }
        uint32_t r[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(acc[i]);
        tmem_st16(tmem_addr(tb, lane_base, C::colS + b * 16), r);
    }
    // d_v 128: K-state of feature t (tile 0) and feature z1f (tile 1), column 0 of each tile
    auto z_init = [&](int f) -> float {
        if (f < 0) return 0.f;
        float acc = 0.f;
        if (from_abi) {
            const short2 ar = s_abi[f];
            if (ar.x >= 0) acc = (ar.y >= 0) ? (zh[ar.x] + zh[ar.y]) * kRsqrt2 : zh[ar.x];
        }
        for (int sp = 0; sp < nprev; ++sp) acc += wsh[(size_t)sp * seg_stride + (size_t)kF * DV + f];
        return acc;
    };
    if (DV == 128 && part == nparts - 1) {
        uint32_t r0[16], r1[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) r0[i] = r1[i] = 0u;
        r0[0] = __float_as_uint(z_init(t));
        r1[0] = __float_as_uint(z_init(z1f));
        tmem_st16(tmem_addr(tb, lane_base, C::colZ0), r0);
        tmem_st16(tmem_addr(tb, lane_base, C::colZ1), r1);
    }
    tmem_wait_st();
}

// ---- the CTA's piece of work: a head, a token range, where its initial state comes from (workspace slots
// ws_first .. ws_first + ws_count - 1) and where its final state goes (slot ws_out, or the caller's state if
// the piece ends its head).
// Legacy grids: blockIdx.x = sequence segment, blockIdx.y = head.
// Balanced grids (one row of CTAs): the concatenation of all heads' chunks, T = heads x chunks per head, is
// cut into n equal ranges [i T / n, (i + 1) T / n), one per SM.  A range holds at most one head boundary
// (n >= heads).  CTA i < n takes range i up to the boundary, if there is one; CTA n + j takes what is left
// of a range behind its boundary, the j-th largest such rest first: the hardware hands these later CTAs to
// SMs as they become free, and the SM whose first piece was shortest is free first, so every SM ends up
// with about T / n chunks.  A piece that ends inside its head leaves its state in slot i of its range.
// A CTA's start-up and wind-down cost as much as `pad` chunks, and an SM with a head boundary pays them twice:
// in this count every head is preceded by `pad` chunks that nobody runs, so such an SM gets that many fewer.
struct Piece { int head, seg, begin, end, first, count, out, head_end, skip; };
// Every thread of the CTA calls it.  find_piece is the same out of line, with the result in shared memory: how this
// arithmetic is compiled into the kernel moves the time of the role loops by several per cent either way (register
// allocation), so each instance of the kernel takes the form that measured faster for it (Cfg::kPieceOutOfLine).
template <int MODE, bool SCAN>
__device__ __forceinline__ void piece_of_cta(Piece& piece, int* s_rest, int balanced, int heads, int pad, int L, int seg_len, int nseg) {
    bool skip = false;
    int it_head = blockIdx.y, it_seg = blockIdx.x, it_begin = blockIdx.x * seg_len, it_end = 0, it_first = 0, it_count = 0,
        it_out = -1;
    bool it_head_end = false;
    if (MODE != kModePre && balanced > 0) {      // (the recompute mode's kernel is never launched this way)
        // 32-bit arithmetic throughout (the host takes this path only while (T + 1) n fits: 64-bit divisions
        // would be subroutine calls, and their mere presence slows this kernel's role loops by a fifth)
        const uint32_t n = balanced;
        const uint32_t nchr = (L + kC - 1) / kC;                // chunks of a head
        const uint32_t w = pad, nchh = nchr + w;                // ... and with the pad in front of them
        const uint32_t T = (uint32_t)heads * nchh;
        uint32_t lo, hi, range;                    // global (padded) chunk range of this piece, index of its range
        if (blockIdx.x < n) {
            range = blockIdx.x;
            lo = range * T / n;
            hi = (range + 1) * T / n;
            const uint32_t xb = ((hi - 1) / nchh) * nchh;         // start of the head that holds the range's last chunk
            if (xb > lo) hi = xb;                                  // a boundary inside: stop there
        } else {
            // rest of the range behind head boundary h: [h nchh, end of the range that holds it); rank the rests
                        const int nb = heads - 1, want = (int)(blockIdx.x - n);
            auto rest_of = [&](uint32_t h, uint32_t& rg) -> int {
                const uint32_t x = h * nchh;
                rg = ((x + 1) * n + T - 1) / T - 1;                 // the range that holds chunk x
                if (rg * T / n == x) return 0;                      // the boundary is a range start
                const uint32_t r = (rg + 1) * T / n - x;
                return r > w ? (int)(r - w) : 0;                    // real chunks behind the pad
            };
            for (int h = 1 + threadIdx.x; h <= nb; h += kThreads) { uint32_t rg; s_rest[h] = rest_of(h, rg); }
            __syncthreads();
            s_rest[0] = -1;
            __syncthreads();
            for (int h = 1 + threadIdx.x; h <= nb; h += kThreads) {
                const int mine = s_rest[h];
                int rank = 0;
                for (int u = 1; u <= nb; ++u) rank += (s_rest[u] > mine || (s_rest[u] == mine && u < h)) ? 1 : 0;
                if (rank == want) s_rest[0] = h;
            }
            __syncthreads();
            const int h = s_rest[0];
            __syncthreads();
            if (h < 1) { skip = true; goto done; }
            const int r = rest_of(h, range);
            if (r == 0) { skip = true; goto done; }               // nothing is left behind this boundary
            lo = (uint32_t)h * nchh;
            hi = lo + w + r;
        }
        it_head = (int)(lo / nchh);
        const uint32_t o0 = lo - (uint32_t)it_head * nchh, o1 = hi - (uint32_t)it_head * nchh;
        const int c0 = (int)(o0 > w ? o0 - w : 0), c1 = (int)(o1 > w ? o1 - w : 0);     // real chunks of the head
        it_seg = c0 > 0 ? 1 : 0;
        it_begin = c0 * kC;
        it_end = min(L, c1 * kC);
        it_head_end = c1 == (int)nchr;
        if (c0 > 0 && MODE != kModeState) {
            if (SCAN) {                            // the slot of the range before: the head's state up to there
                it_first = (int)range - 1;
                it_count = 1;
            } else {                               // every slot of the head so far
                const uint32_t x = (uint32_t)it_head * nchh + w;
                it_first = (int)(((x + 1) * n + T - 1) / T - 1);   // the range that holds the head's first chunk
                it_count = (int)range - it_first;
            }
        }
        if (MODE == kModeState) {
            if (it_head_end) skip = true;                          // nobody starts from the state of a head's last piece
            it_out = (int)range;
        }
    } else {
        it_end = min(L, it_begin + seg_len);
        it_head_end = it_seg == nseg - 1;
        // workspace slots of one head: one per segment but the last, behind (pad = 1) one that holds the caller's
        // state of a continued call (abi_to_slot_kernel), which the segments then take like an earlier segment's
        const int per_head = nseg > 1 ? nseg - 1 + pad : 0;
        const int before = it_seg + pad;                       // slots this segment starts from
        it_first = it_head * per_head + ((SCAN && before > 0) ? before - 1 : 0);
        it_count = (MODE == kModeState || MODE == kModePre || before == 0) ? 0 : (SCAN ? 1 : before);
        it_out = MODE == kModeState ? it_head * per_head + before : -1;
    }
done:
    piece.head = it_head; piece.seg = it_seg; piece.begin = it_begin; piece.end = it_end;
    piece.first = it_first; piece.count = it_count; piece.out = it_out; piece.head_end = it_head_end ? 1 : 0;
    piece.skip = skip ? 1 : 0;
}
template <int MODE, bool SCAN>
__device__ __noinline__ void find_piece(Piece* piece, int* s_rest, int balanced, int heads, int pad, int L, int seg_len, int nseg) {
    Piece pc;
    piece_of_cta<MODE, SCAN>(pc, s_rest, balanced, heads, pad, L, seg_len, nseg);
    __syncthreads();
    if (threadIdx.x == 0) *piece = pc;
    __syncthreads();
}

template <int DV, int MODE>
__global__ void __launch_bounds__(kThreads, 1)
    prefill_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                      const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                      const Params p) {
    using C = Cfg<DV>;
    constexpr int NS = (MODE == kModeState) ? C::kStagesState : C::kStages;
    constexpr bool STATE_ONLY = MODE == kModeState;
    constexpr bool PRE = MODE == kModePre;
    // phi(Q) in tensor memory and two state-copy tiles: the plain chunk loop only (measured: -7 % where every
    // SM has a CTA; the recompute mode's kernel loses 5 % with it)
    constexpr bool PQT = C::kPQinT && MODE == kModeMain;
    // packed bf16 polynomial and the row sums by the tensor cores: the same kernel (measured: -6 % there, +14 % in
    // the recompute mode's kernel)
    constexpr bool PKW = PQT;
    // d_v 128: most of phi(Q) in tensor memory and two output staging tiles (see Cfg::colPQlo)
    constexpr bool PQS = DV == 128 && MODE == kModeMain;
    static_assert(!PQS || C::colPQlo + 48 <= 512, "TMEM budget");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::offMisc);
    uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(bars + kNumBars);
    volatile uint32_t* abort_flag = tmem_base_s + 1;
    float* s_den = reinterpret_cast<float*>(tmem_base_s + 2);          // [4][128] row sums of in-chunk weights
    short2* s_abi = reinterpret_cast<short2*>(s_den + 4 * kC);         // [160] ABI rows of each internal feature

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // ---- the CTA's piece of work (see find_piece)
    Piece pc;
#ifdef BASED_PIECE_OUT
    constexpr bool kPieceOut = (BASED_PIECE_OUT >> ((DV == 128 ? 3 : 0) + MODE)) & 1;
#else
    constexpr bool kPieceOut = DV == 64 && MODE == kModeMain;
#endif
    if constexpr (kPieceOut) {
        Piece* s_piece = reinterpret_cast<Piece*>(s_abi + kF);
        find_piece<MODE, C::kSlotScan>(s_piece, reinterpret_cast<int*>(smem + C::offStage), p.balanced, p.heads, p.pad, p.L, p.seg_len, p.nseg);
        pc = *s_piece;
    } else {
        piece_of_cta<MODE, C::kSlotScan>(pc, reinterpret_cast<int*>(smem + C::offStage), p.balanced, p.heads, p.pad, p.L, p.seg_len, p.nseg);
    }
    if (pc.skip) return;
    const int it_seg = pc.seg, it_head = pc.head, it_begin = pc.begin, it_end = pc.end;
    const int it_first = pc.first, it_count = pc.count, it_out = pc.out;
    const bool it_head_end = pc.head_end != 0;
    const int seg = it_seg, head = it_head, tok_begin = it_begin, tok_end = it_end;
    const int ws_first = it_first, ws_count = it_count, ws_out = it_out;
    const bool head_end = it_head_end;
    const int nch = (tok_end - tok_begin + kC - 1) / kC;
    // Recompute mode: before its own chunks the CTA runs the state update alone ("pre-chunks") over
    // every chunk that precedes its segment.  g counts pre-chunks and own chunks together; stage
    // ring, phi(K) tile and state-update barriers are indexed by g, everything else by c = g - npre.
    const int npre = PRE ? tok_begin / kC : 0;
    const int ntot = npre + nch;
    const int tok_first = tok_begin - npre * kC;

    // shared-memory layout: as in Cfg, except in the state pass (see Cfg::kStagesState)
    constexpr uint32_t kStride = STATE_ONLY ? C::kQKBytes + C::kVBytes : C::kStageBytes;     // bytes of one stage
    constexpr uint32_t kOffK = STATE_ONLY ? 0u : C::kQKBytes, kOffV = kOffK + C::kQKBytes;     // k and v tile within a stage
    constexpr uint32_t offOnesM = STATE_ONLY ? NS * kStride : C::offOnes;
    constexpr uint32_t offPKM = offOnesM + C::kOnesBytes, offPQM = offPKM + C::kPhiBytes;
    static_assert(offPQM + C::kPhiBytes <= C::offMisc && offPKM % 1024 == 0 && kStride % 1024 == 0, "state pass layout");
    uint8_t* sPK = smem + offPKM;
    uint8_t* sPQ = smem + offPQM;
    uint8_t* sSc = smem + C::offSc;
    uint8_t* sOnes = smem + offOnesM;
    uint8_t* sOut = smem + C::offOut;

    if (tid == 0) { TRACE(5, 0, 7); TRACE_CTA(0); }     // kernel entry
    // state pass: the main pass of the same call may be scheduled behind this CTA (see launch_main_after_state)
    if (STATE_ONLY) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(&bars[kFull0 + s], 1); mbar_init(&bars[kEmpty0 + s], STATE_ONLY ? 1 : 2); }
        mbar_init(&bars[kG1], 1); mbar_init(&bars[kG1b], 1); mbar_init(&bars[kPb], 128); mbar_init(&bars[kG2], 1); mbar_init(&bars[kG2b], 1); mbar_init(&bars[kG4], 1); mbar_init(&bars[kG4b], 1);
        mbar_init(&bars[kTR], 128); mbar_init(&bars[kTRb], 128); mbar_init(&bars[kSC], 128); mbar_init(&bars[kSCb], 128);
        mbar_init(&bars[kG3], 1);
        mbar_init(&bars[kP], 128); mbar_init(&bars[kR4], PQT ? 256 : 384); mbar_init(&bars[kPK], 128); mbar_init(&bars[kPKb], 128); mbar_init(&bars[kDone], 1);
        mbar_init(&bars[kSR], 128);
        mbar_init(&bars[kFin], 1);
        mbar_init(&bars[kInit], 384);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v); prefetch_tensormap(&tm_o);
    }
    if (warp == kWarpMma) { tmem_alloc(tmem_base_s, 512); tmem_relinquish(); }
    if (tid < kF) {
        const AbiRows ar = p.sym ? sym_rows(tid) : abi_rows(tid);
        s_abi[tid] = make_short2((short)ar.a, (short)ar.b);
    }
    const int abi_nrows = p.sym ? kDSym : kD;
    // constant operand tiles and a zeroed state-copy tile (its rows past d_v + 1 stay zero for good)
    if (DV == 64) {
        for (uint32_t i = tid * 16; i < C::kOnesBytes; i += kThreads * 16) {
            const uint32_t t = i >> 7, chunk = (i >> 4) & 7;      // token row, 16-byte chunk within the 128-byte row
            const uint32_t first = (chunk == (t & 7)) ? 0x00003F80u : 0u;   // element (t, column 0) = 1.0
            *reinterpret_cast<uint4*>(sOnes + i) = make_uint4(first, 0u, 0u, 0u);
        }
    } else {
        for (uint32_t i = tid * 16; i < C::kOnesBytes; i += kThreads * 16)
            *reinterpret_cast<uint4*>(sOnes + i) = make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
    }
    if (!STATE_ONLY) {
        for (uint32_t i = tid * 16; i < C::kScBytes; i += kThreads * 16)
            *reinterpret_cast<uint4*>(sSc + i) = make_uint4(0u, 0u, 0u, 0u);
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // The recompute-mode kernel is a programmatic dependent launch: a CTA may get here, past its set-up, while the grid
    // before it in the stream still runs.  It waits for that grid to complete before it touches global memory, and
    // only then lets the grid behind it be scheduled (a grid is never scheduled before everything two grids back is
    // complete).  Short calls gain a tenth from it (cfg 2 back to back: 22.9 -> 20.4 us).  Not in the other modes: the
    // same two instructions in the plain chunk loop's kernel cost it 1-4 %.
    if (MODE == kModePre) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }
    const uint32_t tb = *tmem_base_s;
    const uint32_t lane_base = (uint32_t)(warp & 3) * 32u;     // TMEM lanes this warp may touch
    bool ok = true;
    // "State update of chunk c done".  A parity wait can only tell a phase from the one before it,
    // so a waiter may lag its barrier by at most one phase: the state-only pass, whose feature group
    // works two chunks ahead on two alternating tiles, uses one barrier per tile.
    // Scores / weights of chunk c: with two score buffers the row group may run a chunk ahead of the
    // MMA issuer (and the issuer's scores a chunk ahead of the row group), so each buffer has its own pair.
    auto t_idx = [&](int c) -> int { return C::kTDouble ? (c & 1) : 0; };
    auto t_parity = [&](int c) -> uint32_t { return C::kTDouble ? ((c >> 1) & 1) : (c & 1); };
    // The state-only pass and the pre-chunks alternate between two phi(K) tiles (the phi(Q) tile is
    // free there), even chunks on kG2, odd ones on kG2b; own chunks of the main pass use kG2 alone,
    // continuing its phase count after the even pre-chunks.
    auto alt = [&](int g) -> bool { return STATE_ONLY || g < npre; };
    auto g2_bar = [&](int g) -> uint64_t* { return &bars[(alt(g) && (g & 1)) ? kG2b : kG2]; };
    auto g2_parity = [&](int g) -> uint32_t {
        return alt(g) ? ((g >> 1) & 1) : (uint32_t)(((npre + 1) >> 1) + (g - npre)) & 1u;
    };
    // "phi(K) of chunk g written": one barrier per tile for the same reason (the feature group may be
    // two chunks ahead of the issuer where tiles alternate); same phase numbering as above
    auto pk_bar = [&](int g) -> uint64_t* { return &bars[(alt(g) && (g & 1)) ? kPKb : kPK]; };
    // "step (4) of own chunk c done": with two state-copy tiles (kPQinT) one barrier per tile, as above
    auto g4_bar = [&](int c) -> uint64_t* { return &bars[(PQT && (c & 1)) ? kG4b : kG4]; };
    auto g4_parity = [&](int c) -> uint32_t { return PQT ? ((c >> 1) & 1) : (c & 1); };

    // ---- initial state from earlier pieces' slots, d_v 128 (see Cfg::kSlotScan): in the main pass behind a state pass
    // all four role groups share it
    const bool share_init = !C::kSlotScan && MODE == kModeMain && ws_count > 0;
    auto init_state = [&](int part, int nparts) {
        init_state_blocks<DV>(p.ws + (size_t)ws_first * seg_state_floats(DV), ws_count, MODE == kModeMain && ws_count > 0,
                              (!STATE_ONLY && p.continue_abi) ? p.kv_abi : nullptr, p.z_abi, p.dv, head * abi_nrows, s_abi, tb,
                              part, nparts);
    };
    if constexpr (!C::kSlotScan) {
        if (share_init && warp < 16 && (warp >> 2) != 2) {      // row, feature and output group (parts 0, 1, 3)
            init_state(warp >> 2, 4);
            tc_fence_before();
            mbar_arrive(&bars[kInit]);
        }
    }

    if (warp == kWarpTma) {
        // ===================================================================== TMA producer
        if (lane == 0) {
            for (int g = 0; g < ntot && ok; ++g) {
                const int s = g % NS;
                ok = mbar_wait(&bars[kEmpty0 + s], ((g / NS) & 1) ^ 1, abort_flag);
                if (!ok) break;
                TRACE(1, g, 3);
                uint8_t* st = smem + C::offStage + s * kStride;
                const int tok0 = tok_first + g * kC;
                const bool with_q = !STATE_ONLY && g >= npre;
                mbar_arrive_expect_tx(&bars[kFull0 + s], (with_q ? 2 : 1) * C::kQKBytes + C::kVBytes);
                if (with_q) tma_load_3d(st, &tm_q, &bars[kFull0 + s], 0, tok0, head);
                tma_load_3d(st + kOffK, &tm_k, &bars[kFull0 + s], 0, tok0, head);
#pragma unroll
                for (int b = 0; b < DV / 64; ++b)
                    tma_load_3d(st + kOffV + b * (kC * 128), &tm_v, &bars[kFull0 + s], b * 64, tok0, head);
            }
        }
    } else if (warp == kWarpMma) {
        // ===================================================================== MMA issuer, state chain
        // (the whole warp runs the loop and one elected lane issues: see mma_ss_w)
        const uint32_t lead = elect_one();
        {
            constexpr uint64_t dPhiMN = make_smem_desc_base(C::kPhiBlk, 512, kSwizzle64B);// MN-major view of a phi tile
            constexpr uint64_t dV = make_smem_desc_base(kC * 128, 1024, kSwizzle128B);    // MN-major [128 tok][DV]
            constexpr uint64_t dOnes = make_smem_desc_base(16, 1024, kSwizzle128B);
            constexpr uint32_t iZ0 = make_idesc_bf16(128, 16, 1, 0);
            constexpr uint32_t iZ1 = make_idesc_bf16(64, 16, 1, 0);
            constexpr uint32_t i5 = make_idesc_bf16(128, kF, 1, 1);
            const uint32_t aOnes = smem_u32(sOnes);
            const uint32_t lV = desc_lo(dV), lOnes = desc_lo(dOnes) + (aOnes >> 4);
            // STATE_ONLY alternates between two phi(K) tiles (the phi(Q) tile is unused there)
            const uint32_t lPK0 = desc_lo(dPhiMN) + (smem_u32(sPK) >> 4), lPK1 = desc_lo(dPhiMN) + (smem_u32(sPQ) >> 4);
            for (int c = 0; c < ntot && ok; ++c) {      // c counts pre-chunks and own chunks here
                const int s = c % NS;
                const uint32_t aVt = smem_u32(smem + C::offStage + s * kStride) + kOffV;
                const uint32_t lPK = (alt(c) && (c & 1)) ? lPK1 : lPK0;
                ok = mbar_wait(&bars[kFull0 + s], (c / NS) & 1, abort_flag);
                if (ok) ok = mbar_wait(pk_bar(c), g2_parity(c), abort_flag);
                // the state group has read (or, before the first chunk, initialised) the state in TMEM:
                // phase 0 of the barrier is the initialisation when there are pre-chunks (or in the
                // state-only pass), and own chunk i is phase i (+1 after pre-chunks)
                if (ok) {
                    if (STATE_ONLY || c < npre) {
                        if (c == 0) ok = mbar_wait(&bars[kSR], 0, abort_flag);
                    } else {
                        ok = mbar_wait(&bars[kSR], (uint32_t)(c - npre + (npre > 0 ? 1 : 0)) & 1u, abort_flag);
                    }
                }
                if (!ok) break;
                if (lane == 0) TRACE(1, c, 1);
                tc_fence_after();
                if (DV == 64) {
                    // V^T as a 128-row A operand: rows 0..63 from the V tile, rows 64..127 from the ones
                    // block (row 64 = ones over the tokens), so lane 64 of S^T accumulates z
                    const uint64_t dV1 = make_smem_desc_base(aOnes - aVt, 1024, kSwizzle128B);
                    const uint32_t a_lo = desc_lo(dV1) + (aVt >> 4), a_hi = desc_hi(dV1);
#pragma unroll
                    for (int k = 0; k < kC / 16; ++k)         // (start + 2 KB per K-step, block offset - 2 KB: see kOnesBytes)
                        mma_ss_w<true>(lead, tb + C::colS, a_lo + k * ((2048u >> 4) - ((2048u >> 4) << 16)), a_hi,
                                       lPK + k * (1024 >> 4), desc_hi(dPhiMN), i5);
                } else {
                    const uint32_t a_lo = lV + (aVt >> 4);
#pragma unroll
                    for (int k = 0; k < kC / 16; ++k) {
                        mma_ss_w<true>(lead, tb + C::colS, a_lo + k * (2048 >> 4), desc_hi(dV), lPK + k * (1024 >> 4),
                                        desc_hi(dPhiMN), i5);
                        mma_ss_w<true>(lead, tb + C::colZ0, lPK + k * (1024 >> 4), desc_hi(dPhiMN), lOnes + (k & 1) * 2,
                                        desc_hi(dOnes), iZ0);
                        mma_ss_w<true>(lead, tb + C::colZ1, lPK + ((4 * C::kPhiBlk + k * 1024) >> 4), desc_hi(dPhiMN),
                                        lOnes + (k & 1) * 2, desc_hi(dOnes), iZ1);
                    }
                }
                mma_commit_w(lead, g2_bar(c));
                mma_commit_w(lead, &bars[kEmpty0 + s]);
                // every state update without a read-out in between is done (state-only pass: all of
                // them; main pass: the pre-chunks)
                if (c + 1 == (STATE_ONLY ? nch : npre)) mma_commit_w(lead, &bars[kDone]);
                if (c + 1 == ntot) mma_commit_w(lead, &bars[kFin]);      // the state is final
                if (lane == 0) TRACE(1, c, 2);
            }
        }
    } else if (warp == kWarpMmaY) {
        // ===================================================================== MMA issuer, output chain
        const uint32_t lead = elect_one();
        if (!STATE_ONLY) {
            constexpr uint64_t dQK = make_smem_desc_base(16, 256, kSwizzle32B);           // K-major [128][16]
            constexpr uint64_t dPhiK = make_smem_desc_base(16, 512, kSwizzle64B);         // K-major, 64-byte rows
            constexpr uint64_t dV = make_smem_desc_base(kC * 128, 1024, kSwizzle128B);    // MN-major [128 tok][DV]
            constexpr uint32_t i1 = make_idesc_bf16(128, 128, 0, 0);
            constexpr uint32_t i4 = make_idesc_bf16(128, C::kNY, 0, 0);
            // d_v 64, plain chunk loop: the values get 16 more columns from the ones block (column 64 = 1 for every token), so the same
            // MMAs that apply the weights to V also add up each row's weights: the in-chunk part of the denominator
            // lands in column 64 of Y, on top of the cross-chunk part that step (4) put there
            constexpr uint32_t i3 = make_idesc_bf16(128, PKW ? DV + 16 : DV, 0, 1);
            const uint32_t lQK = desc_lo(dQK), lV = desc_lo(dV);
            const uint32_t lPQ = desc_lo(dPhiK) + (smem_u32(sPQ) >> 4), lSc0 = desc_lo(dPhiK) + (smem_u32(sSc) >> 4);
            // scores of chunk c: T[c & 1] (or the single T) = Q_c K_c^T
            auto issue_scores = [&](int c) -> bool {
                const int s = (c + npre) % NS;
                if (!mbar_wait(&bars[kFull0 + s], ((c + npre) / NS) & 1, abort_flag)) return false;
                if (lane == 0) TRACE(0, c, 0);
                tc_fence_after();
                const uint32_t aSt = smem_u32(smem + C::offStage + s * C::kStageBytes);
                mma_ss_w<false>(lead, tb + C::colT + (C::kTDouble ? (c & 1) * 128 : 0), lQK + (aSt >> 4), desc_hi(dQK),
                                 lQK + ((aSt + C::kQKBytes) >> 4), desc_hi(dQK), i1);
                mma_commit_w(lead, &bars[kG1 + t_idx(c)]);
                return true;
            };
            // pre-chunks: nothing to issue, but the stage is released by two arrivals
            for (int g = 0; g < npre && ok; ++g) {
                ok = mbar_wait(&bars[kFull0 + g % NS], (g / NS) & 1, abort_flag);
                if (ok && lead) mbar_arrive(&bars[kEmpty0 + g % NS]);
            }
            if (nch > 0 && ok) ok = issue_scores(0);
            for (int c = 0; c < nch && ok; ++c) {
                const int s = (c + npre) % NS;
                const uint32_t ph = c & 1;
                const uint32_t aVt = smem_u32(smem + C::offStage + s * C::kStageBytes) + 2 * C::kQKBytes;
                const uint32_t colTc = C::colT + (C::kTDouble ? (c & 1) * 128 : 0);
                // with two score buffers the next chunk's scores are issued ahead of this chunk's
                // steps (4) and (3), so its polynomial overlaps them
                if (lane == 0) TRACE(2, c, 3);
                if (C::kTDouble && c + 1 < nch) {
                    ok = issue_scores(c + 1);
                    if (!ok) break;
                }
                if (lane == 0) TRACE(0, c, 1);
                // step (4) of chunk c needs phi(Q) of chunk c (feature group), the state copy after chunk
                // c-1 (state group) and the Y accumulator read out for chunk c-1 (output group, which
                // arrives once before its first chunk): one barrier, three groups of 128 arrivals
                ok = mbar_wait(&bars[kR4], ph, abort_flag);
                if (!ok) break;
                // two copy tiles: the state group may be a chunk ahead, so its "copy written" has a barrier per tile
                if (PQT) {
                    ok = mbar_wait(&bars[kSC + (c & 1)], (c >> 1) & 1, abort_flag);
                    if (!ok) break;
                }
                if (lane == 0) TRACE(0, c, 3);
                tc_fence_after();
                const uint32_t lSc = (PQT && (c & 1)) ? lPQ : lSc0;      // second copy tile: the phi(Q) tile's place
#pragma unroll
                for (int k = 0; k < kF / 16; ++k) {
                    const uint32_t off = ((k >> 1) * C::kPhiBlk + (k & 1) * 32) >> 4;
                    const uint32_t offb = ((k >> 1) * C::kScBlk + (k & 1) * 32) >> 4;
                    if (PQT) {
                        const uint32_t a = tb + (k < 8 ? colTc + 64 + k * 8 : C::colPQhi + (k - 8) * 8);
                        if (k == 0) mma_ts_w<false>(lead, tb + C::colY, a, lSc + offb, desc_hi(dPhiK), i4);
                        else mma_ts_w<true>(lead, tb + C::colY, a, lSc + offb, desc_hi(dPhiK), i4);
                    } else if (PQS) {
                        const uint32_t offs = (((k >> 1) - 3) * C::kPhiBlk + (k & 1) * 32) >> 4;      // blocks 3, 4 at the tile's start
                        if (k == 0) mma_ts_w<false>(lead, tb + C::colY, tb + C::colPQlo, lSc + offb, desc_hi(dPhiK), i4);
                        else if (k < 6) mma_ts_w<true>(lead, tb + C::colY, tb + C::colPQlo + k * 8, lSc + offb, desc_hi(dPhiK), i4);
                        else mma_ss_w<true>(lead, tb + C::colY, lPQ + offs, desc_hi(dPhiK), lSc + offb, desc_hi(dPhiK), i4);
                    } else {
                        if (k == 0) mma_ss_w<false>(lead, tb + C::colY, lPQ + off, desc_hi(dPhiK), lSc + offb, desc_hi(dPhiK), i4);
                        else mma_ss_w<true>(lead, tb + C::colY, lPQ + off, desc_hi(dPhiK), lSc + offb, desc_hi(dPhiK), i4);
                    }
                }
                mma_commit_w(lead, g4_bar(c));
                if (lane == 0) TRACE(0, c, 4);
                ok = mbar_wait(&bars[kP + t_idx(c)], t_parity(c), abort_flag);
                if (!ok) break;
                if (lane == 0) TRACE(0, c, 5);
                tc_fence_after();
                {
                    // there the second 64-column block of the B operand is the ones block (leading byte offset)
                    const uint64_t dVo = PKW ? make_smem_desc_base(smem_u32(sOnes) - aVt, 1024, kSwizzle128B) : dV;
                    const uint32_t b_lo = desc_lo(dVo) + (aVt >> 4), b_hi = desc_hi(dVo);
#pragma unroll
                    for (int k = 0; k < kC / 16; ++k)
                        mma_ts_w<true>(lead, tb + C::colY, tb + colTc + k * 8,
                                       b_lo + k * (PKW ? (2048u >> 4) - ((2048u >> 4) << 16) : (2048u >> 4)), b_hi, i3);
                }
                if (lane == 0) TRACE(2, c, 2);
                mma_commit_w(lead, &bars[kG3]);
                mma_commit_w(lead, &bars[kEmpty0 + s]);
                if (lane == 0) TRACE(0, c, 6);
                // single score buffer: P of this chunk has to be consumed before the next scores land
                if (!C::kTDouble && c + 1 < nch) ok = issue_scores(c + 1);
            }
        }
    } else if (warp >= 12) {
        // ===================================================================== output group
        // One thread per output row: Y / (row sum + cross-chunk denominator + eps) -> bf16 ->
        // swizzled staging tile of 64 columns -> TMA store.
        if (!STATE_ONLY) {
            const int t = tid - 384;
            uint8_t* orow = sOut + (t >> 3) * 1024 + (t & 7) * 128;
            const uint32_t sw = t & 7;
            if (nch > 0) mbar_arrive(&bars[kR4]);            // the Y accumulator starts out free
            for (int c = 0; c < nch && ok; ++c) {
                ok = group_all(1, mbar_wait(&bars[kG3], c & 1, abort_flag));
                if (!ok) break;
                if (t == 0) TRACE(5, c, 0);
                tc_fence_after();
                uint32_t dcol;
                tmem_ld1(tmem_addr(tb, lane_base, C::colY + DV), dcol);
                tmem_wait_ld();
                const float den_in = PKW ? 0.f : s_den[(c & 3) * kC + t];      // packed variant: already in the column
                const float inv = p.numerator_only ? 1.0f : 1.0f / (den_in + __uint_as_float(dcol) + kEps);
                if constexpr (PQS) {
                    // All of Y leaves tensor memory before any staging (step (4) of the next chunk waits for that), 32
                    // columns at a time, scaled and packed as they arrive: 128 fp32 columns do not fit a thread's registers.
                    // Then one staging tile per 64 columns: a bulk store reads its tile at about 15 bytes per cycle, so
                    // with one tile filled and drained twice per chunk the tile alone would take most of a chunk's time.
                    uint32_t pkd[DV / 2];
#pragma unroll
                    for (int qd = 0; qd < DV / 32; ++qd) {
                        uint32_t y[32];
                        tmem_ld32(tmem_addr(tb, lane_base, C::colY + qd * 32), y);
                        tmem_wait_ld();
                        if (qd == DV / 32 - 1) {
                            tc_fence_before();
                            mbar_arrive(&bars[kR4]);
                            if (t == 0) TRACE(5, c, 1);
                        }
                        const uint64_t inv2 = f32x2(__float_as_uint(inv), __float_as_uint(inv));
#pragma unroll
                        for (int i = 0; i < 16; ++i) pkd[qd * 16 + i] = scale_pack(y[2 * i], y[2 * i + 1], inv2);
                    }
#pragma unroll
                    for (int h = 0; h < DV / 64; ++h) {
                        uint8_t* tile = h == 0 ? sOut : smem + C::offOut2;
                        uint8_t* trow = tile + (t >> 3) * 1024 + (t & 7) * 128;
                        // the tile is free once the store before the latest one has read it
                        if (t == 0) tma_store_wait_read<1>();
                        group_sync(1);
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            *reinterpret_cast<uint4*>(trow + ((j ^ sw) << 4)) =
                                make_uint4(pkd[h * 32 + 4 * j], pkd[h * 32 + 4 * j + 1], pkd[h * 32 + 4 * j + 2], pkd[h * 32 + 4 * j + 3]);
                        fence_proxy_async_smem();
                        group_sync(1);
                        if (t == 0) {
                            tma_store_3d(&tm_o, tile, h * 64, tok_begin + c * kC, head);   // rows past the end are clipped
                            tma_store_commit();
                        }
                    }
                } else {
#pragma unroll 1
                for (int h = 0; h < DV / 64; ++h) {
                    uint32_t y0[32], y1[32];
                    tmem_ld32(tmem_addr(tb, lane_base, C::colY + h * 64), y0);
                    tmem_ld32(tmem_addr(tb, lane_base, C::colY + h * 64 + 32), y1);
                    tmem_wait_ld();
                    if (h == DV / 64 - 1) {            // all of Y is in registers: release the accumulator
                        tc_fence_before();
                        mbar_arrive(&bars[kR4]);
                        if (t == 0) TRACE(5, c, 1);
                    }
                    // the staging tile is free once the previous TMA store has read it
                    if (t == 0) tma_store_wait_read<0>();
                    group_sync(1);
                    const uint64_t inv2 = f32x2(__float_as_uint(inv), __float_as_uint(inv));
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        *reinterpret_cast<uint4*>(orow + ((j ^ sw) << 4)) =
                            make_uint4(scale_pack(y0[8 * j], y0[8 * j + 1], inv2), scale_pack(y0[8 * j + 2], y0[8 * j + 3], inv2),
                                       scale_pack(y0[8 * j + 4], y0[8 * j + 5], inv2), scale_pack(y0[8 * j + 6], y0[8 * j + 7], inv2));
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        *reinterpret_cast<uint4*>(orow + (((4 + j) ^ sw) << 4)) =
                            make_uint4(scale_pack(y1[8 * j], y1[8 * j + 1], inv2), scale_pack(y1[8 * j + 2], y1[8 * j + 3], inv2),
                                       scale_pack(y1[8 * j + 4], y1[8 * j + 5], inv2), scale_pack(y1[8 * j + 6], y1[8 * j + 7], inv2));
                    fence_proxy_async_smem();
                    group_sync(1);
                    if (t == 0) {
                        // rows past the end of the sequence are clipped by the tensor map
                        tma_store_3d(&tm_o, sOut, h * 64, tok_begin + c * kC, head);
                        tma_store_commit();
                    }
                }
                }
                if (t == 0) TRACE(5, c, 2);
            }
            // the staging tile must outlive the last store's read of it; the global writes complete on their own
            if (t == 0) tma_store_wait_read<0>();
        }
    } else if (warp >= 8) {
        // ===================================================================== state group
        // One thread per TMEM lane of the state accumulator: initial state, per-chunk bf16
        // copy of the state for step (4), final state.
        const int t = tid - 256;
        // what this thread's lane of S^T holds: V column srow, or (d_v 64) the K-state at lane 64
        const int srow = (t < C::kSLanes) ? t : -1;
        const bool is_z = (DV == 64) && t == 64;
        // d_v 128: K-state features held in the two z tiles (64-row MMA: rows 0..31 in lanes 0-15, 32-47)
        const int z1f = (DV == 128 && (t & 31) < 16 && (t >> 5) < 2) ? 128 + (t >> 5) * 16 + (t & 15) : -1;
        if constexpr (C::kSlotScan) {
            const size_t seg_stride = seg_state_floats(DV);
            const float* wsh = p.ws + (size_t)ws_first * seg_stride;      // the partial states this piece starts from
            const int dv = p.dv;                        // row pitch of the caller's state; lanes >= dv hold zeros
            const float* kvh = p.kv_abi ? p.kv_abi + (size_t)head * abi_nrows * dv : nullptr;
            const float* zh = p.z_abi ? p.z_abi + (size_t)head * abi_nrows : nullptr;
            const bool from_abi = !STATE_ONLY && p.continue_abi;
            const int nprev = ws_count;
            // the partial states are the state pass's output (a no-op when this grid was launched the plain way)
            if (MODE == kModeMain && nprev > 0) asm volatile("griddepcontrol.wait;" ::: "memory");

            // Initial value of this lane's row: the caller's ABI state (folded into the internal
            // basis) plus the partial states of the earlier segments.  Loads are issued 16 at a
            // time before they are consumed, so their latencies overlap.
#pragma unroll 1
            for (int b = 0; b < kF / 16; ++b) {
                float acc[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[i] = 0.f;
                if (srow >= 0) {
                    if (from_abi) {
                        float va[16], vb[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const short2 ar = s_abi[b * 16 + i];
                            const bool live = is_z || srow < dv;
                            va[i] = (ar.x >= 0 && live) ? (is_z ? zh[ar.x] : kvh[(size_t)ar.x * dv + srow]) : 0.f;
                            vb[i] = (ar.y >= 0 && live) ? (is_z ? zh[ar.y] : kvh[(size_t)ar.y * dv + srow]) : 0.f;
                        }
#pragma unroll
                        for (int i = 0; i < 16; ++i) acc[i] = (s_abi[b * 16 + i].y >= 0) ? (va[i] + vb[i]) * kRsqrt2 : va[i];
                    }
                    for (int sp = 0; sp < nprev; ++sp) {
                        const float* src = wsh + (size_t)sp * seg_stride + (is_z ? (size_t)kF * DV + b * 16
                                                                                 : (size_t)(b * 16) * DV + srow);
                        float tmp[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) tmp[i] = is_z ? src[i] : src[(size_t)i * DV];
#pragma unroll
                        for (int i = 0; i < 16; ++i) acc[i] += tmp[i];
                    }
                }
                uint32_t r[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(acc[i]);
                tmem_st16(tmem_addr(tb, lane_base, C::colS + b * 16), r);
            }
            // d_v 128: K-state of feature t (tile 0) and feature z1f (tile 1), column 0 of each tile
            auto z_init = [&](int f) -> float {
                if (f < 0) return 0.f;
                float acc = 0.f;
                if (from_abi) {
                    const short2 ar = s_abi[f];
                    if (ar.x >= 0) acc = (ar.y >= 0) ? (zh[ar.x] + zh[ar.y]) * kRsqrt2 : zh[ar.x];
                }
                for (int sp = 0; sp < nprev; ++sp) acc += wsh[(size_t)sp * seg_stride + (size_t)kF * DV + f];
                return acc;
            };
            if (DV == 128) {
                uint32_t r0[16], r1[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) r0[i] = r1[i] = 0u;
                r0[0] = __float_as_uint(z_init(t));
                r1[0] = __float_as_uint(z_init(z1f));
                tmem_st16(tmem_addr(tb, lane_base, C::colZ0), r0);
                tmem_st16(tmem_addr(tb, lane_base, C::colZ1), r1);
            }
        } else if (share_init) {
            init_state(2, 4);
            ok = mbar_wait(&bars[kInit], 0, abort_flag);          // the other groups' blocks are written
            tc_fence_after();
        } else {
            init_state(0, 1);
        }
        tmem_wait_st();
        if (t == 0) TRACE(5, 2, 7);   // state initialised

        if (STATE_ONLY) {
            tc_fence_before();
            mbar_arrive(&bars[kSR]);
            if (nch > 0) ok = mbar_wait(&bars[kDone], 0, abort_flag);
        } else {
            if (npre > 0) {
                tc_fence_before();
                mbar_arrive(&bars[kSR]);                                   // the state is initialised
                ok = mbar_wait(&bars[kDone], 0, abort_flag);               // all pre-chunks are folded in
            }
            for (int c = 0; c < nch && ok; ++c) {
                if (c > 0) {
                    ok = mbar_wait(g2_bar(c + npre - 1), g2_parity(c + npre - 1), abort_flag);   // state after chunk c-1 is final
                    if (!ok) break;
                }
                if (t == 0) TRACE(4, c, 0);
                tc_fence_after();
                // bf16 copy of this lane's state row, held in registers until the tile is free
                uint32_t pkd[kF / 2];
                // d_v 64: lanes 65..127 of S^T hold nothing, so the group's last warp (lanes 96..127) has no row to
                // copy: it only keeps the barriers' arrival counts whole
                if (DV == 128 || t < 96) {
#pragma unroll
                    for (int b = 0; b < kF / 16; ++b) {
                        uint32_t r[16];
                        tmem_ld16(tmem_addr(tb, lane_base, C::colS + b * 16), r);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            pkd[b * 8 + i] = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
                    }
                }
                uint32_t z0 = 0, z1 = 0;
                if (DV == 128) {
                    tmem_ld1(tmem_addr(tb, lane_base, C::colZ0), z0);
                    tmem_ld1(tmem_addr(tb, lane_base, C::colZ1), z1);
                    tmem_wait_ld();
                }
                tc_fence_before();
                mbar_arrive(&bars[kSR]);                                   // step (5) of chunk c may overwrite the state
                if (t == 0) TRACE(4, c, 1);
                // the tile's last reader: step (4) of chunk c-1, or of chunk c-2 where two tiles alternate
                constexpr int kBack = PQT ? 2 : 1;
                if (c >= kBack) {
                    ok = mbar_wait(g4_bar(c - kBack), g4_parity(c - kBack), abort_flag);
                    if (!ok) break;
                }
                if (t == 0) TRACE(4, c, 2);
                uint8_t* sScC = (PQT && (c & 1)) ? sPQ : sSc;
                if (srow >= 0) {
                    uint8_t* row = sScC + (srow >> 3) * 512 + (srow & 7) * 64;
                    const uint32_t sw = (srow >> 1) & 3;
#pragma unroll
                    for (int j = 0; j < kF / 8; ++j)
                        *reinterpret_cast<uint4*>(row + (j >> 2) * C::kScBlk + (((j & 3) ^ sw) << 4)) =
                            make_uint4(pkd[4 * j], pkd[4 * j + 1], pkd[4 * j + 2], pkd[4 * j + 3]);
                }
                if (DV == 128) {
                    // z row (row 128 of the tile: its swizzle term is zero)
                    uint8_t* zrow = sScC + (DV >> 3) * 512;
                    *reinterpret_cast<__nv_bfloat16*>(zrow + (t >> 5) * C::kScBlk + (t & 31) * 2) =
                        __float2bfloat16_rn(__uint_as_float(z0));
                    if (z1f >= 0)
                        *reinterpret_cast<__nv_bfloat16*>(zrow + (uint32_t)(z1f >> 5) * C::kScBlk + (uint32_t)(z1f & 31) * 2) =
                            __float2bfloat16_rn(__uint_as_float(z1));
                }
                fence_proxy_async_smem();
                mbar_arrive(&bars[PQT ? kSC + (c & 1) : kR4]);
                if (t == 0) TRACE(4, c, 3);
            }
            if (ok && nch > 0) ok = mbar_wait(g2_bar(ntot - 1), g2_parity(ntot - 1), abort_flag);
        }

        if (t == 0) TRACE(5, 3, 7);   // chunk loop done
    } else if (warp >= 4) {
        // ===================================================================== feature group
        // One thread per token of the chunk: expands its k row (and q row) into feature rows.
        const int t = tid - 128;
        for (int g = 0; g < ntot && ok; ++g) {
            const int c = g - npre;                     // own chunk index (negative: pre-chunk)
            const int s = g % NS;
            const uint8_t* st = smem + C::offStage + s * kStride;
            const bool valid = tok_first + g * kC + t < tok_end;
            ok = mbar_wait(&bars[kFull0 + s], (g / NS) & 1, abort_flag);
            if (!ok) break;
            if (t == 0) TRACE(3, c, 0);
            uint4 klo, khi, qlo = make_uint4(0u, 0u, 0u, 0u), qhi = qlo;
            read_qk_row(st + kOffK, t, klo, khi);
            if (!STATE_ONLY && c >= 0) read_qk_row(st, t, qlo, qhi);
            // the tile being overwritten was last read by step (5) of the chunk before (two chunks
            // before where tiles alternate; own chunk 0 after pre-chunks: the last even pre-chunk)
            {
                int last = -1;
                if (alt(g)) last = g - 2;
                else if (c > 0) last = g - 1;
                else if (npre > 0) last = (npre - 1) & ~1;
                if (last >= 0) {
                    ok = mbar_wait(g2_bar(last), g2_parity(last), abort_flag);
                    if (!ok) break;
                }
            }
            if (t == 0) TRACE(3, c, 1);
            write_phi_row(klo, khi, (alt(g) && (g & 1)) ? sPQ : sPK, t, valid);
            fence_proxy_async_smem();
            mbar_arrive(pk_bar(g));
            if (t == 0) TRACE(3, c, 2);
            if (!STATE_ONLY && c >= 0) {
                // d_v 64: expand the q row before waiting for the tile, so that only the stores follow the
                // wait (measured: 5 % on the 360M-layer shape; at d_v 128 it costs 1 %, so not there)
                uint4 fq[DV == 64 ? 20 : 1];
                if constexpr (DV == 64) compute_phi_row(qlo, qhi, true, fq);
                if constexpr (PQT) {
                    // the row group has read the scores of chunk c: the upper half of their buffer is free
                    ok = mbar_wait(&bars[kTR + t_idx(c)], t_parity(c), abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t colTc = C::colT + (c & 1) * 128;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t r[16] = {fq[4 * j].x, fq[4 * j].y, fq[4 * j].z, fq[4 * j].w,
                                                fq[4 * j + 1].x, fq[4 * j + 1].y, fq[4 * j + 1].z, fq[4 * j + 1].w,
                                                fq[4 * j + 2].x, fq[4 * j + 2].y, fq[4 * j + 2].z, fq[4 * j + 2].w,
                                                fq[4 * j + 3].x, fq[4 * j + 3].y, fq[4 * j + 3].z, fq[4 * j + 3].w};
                        tmem_st16(tmem_addr(tb, lane_base, colTc + 64 + j * 16), r);
                    }
                }
                if (c > 0) {
                    ok = mbar_wait(g4_bar(c - 1), g4_parity(c - 1), abort_flag);   // step (4) of chunk c-1 has read phi(Q)
                    if (!ok) break;
                } else if (npre > 1) {
                    const int last = ((npre & 1) ? npre - 2 : npre - 1);   // last odd pre-chunk used this tile for phi(K)
                    ok = mbar_wait(g2_bar(last), g2_parity(last), abort_flag);
                    if (!ok) break;
                }
                if (t == 0) TRACE(3, c, 3);
                if constexpr (PQT) {
                    tc_fence_after();
                    const uint32_t r[16] = {fq[16].x, fq[16].y, fq[16].z, fq[16].w, fq[17].x, fq[17].y, fq[17].z, fq[17].w,
                                            fq[18].x, fq[18].y, fq[18].z, fq[18].w, fq[19].x, fq[19].y, fq[19].z, fq[19].w};
                    tmem_st16(tmem_addr(tb, lane_base, C::colPQhi), r);
                    tmem_wait_st();
                    tc_fence_before();
                } else if constexpr (PQS) {
                    // block by block, each stored as it is formed (twenty pieces at once do not fit the registers)
                    uint32_t E[8], O[8], vv[16];
                    phi_prepare(qlo, qhi, true, E, O);
                    tc_fence_after();
                    phi_block<0>(E, O, true, vv); tmem_st16(tmem_addr(tb, lane_base, C::colPQlo), vv);
                    phi_block<1>(E, O, true, vv); tmem_st16(tmem_addr(tb, lane_base, C::colPQlo + 16), vv);
                    phi_block<2>(E, O, true, vv); tmem_st16(tmem_addr(tb, lane_base, C::colPQlo + 32), vv);
                    uint8_t* row = sPQ + (t >> 3) * 512 + (t & 7) * 64;     // feature blocks 3 and 4 -> blocks 0 and 1 of the tile
                    const uint32_t sw = (t >> 1) & 3;
                    phi_block<3>(E, O, true, vv);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        *reinterpret_cast<uint4*>(row + ((j ^ sw) << 4)) = make_uint4(vv[4 * j], vv[4 * j + 1], vv[4 * j + 2], vv[4 * j + 3]);
                    phi_block<4>(E, O, true, vv);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        *reinterpret_cast<uint4*>(row + kC * 64 + ((j ^ sw) << 4)) = make_uint4(vv[4 * j], vv[4 * j + 1], vv[4 * j + 2], vv[4 * j + 3]);
                    tmem_wait_st();
                    tc_fence_before();
                    fence_proxy_async_smem();
                } else {
                    if constexpr (DV == 64) store_phi_row(fq, sPQ, t);
                    else write_phi_row(qlo, qhi, sPQ, t, true);
                    fence_proxy_async_smem();
                }
                mbar_arrive(&bars[kR4]);
                if (t == 0) TRACE(3, c, 4);
            }
        }
    } else if (!STATE_ONLY) {
        // ===================================================================== row group
        // One thread per query row: polynomial of the scores, causal mask, row sum; the
        // bf16 weights overwrite the scores in place (columns [0, 64) of the same lanes).
        const int q4 = warp;                            // lane quarter == 32-row block of the chunk
        // packed variant: causal mask of the batch that holds the diagonal, one word per pair of columns
        // (columns 2i and 2i+1 against this row, i.e. this lane), so that masking is one logic instruction per pair
        uint32_t dm[PKW ? 16 : 1];
        if constexpr (PKW) {
#pragma unroll
            for (int i = 0; i < 16; ++i) dm[i] = (2 * i + 1 <= lane) ? 0xFFFFFFFFu : ((2 * i <= lane) ? 0x0000FFFFu : 0u);
        }
        // sixteen registers of zeros for the batches right of the diagonal (opaque, or each store would be
        // preceded by sixteen moves)
        uint32_t zz[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) asm volatile("mov.b32 %0, 0;" : "=r"(zz[i]));
        for (int c = 0; c < nch && ok; ++c) {
            ok = mbar_wait(&bars[kG1 + t_idx(c)], t_parity(c), abort_flag);
            if (!ok) break;
            if (tid == 96) TRACE(2, c, 0);
            tc_fence_after();
            const uint32_t colTc = C::colT + (C::kTDouble ? (c & 1) * 128 : 0);
            float den0 = 0.f, den1 = 0.f;
#pragma unroll 1
            for (int b = 0; b < 4; ++b) {
                uint32_t pk[16];
                if (b <= q4) {                           // some row of this warp sees these key columns
                    uint32_t sc[32];
                    tmem_ld32(tmem_addr(tb, lane_base, colTc + b * 32), sc);
                    tmem_wait_ld();
                    if constexpr (PKW) {
                        // Two scores per instruction: the pair is rounded to bf16 first, w = 1 + s (1/4 + s/32) in
                        // two packed fused multiply-adds, and the result is the packed weight as it is stored (it
                        // would be rounded to bf16 anyway).  The row sum is the tensor cores' work (see step (3)).
                        const __nv_bfloat162 c1 = __float2bfloat162_rn(0.25f), c2 = __float2bfloat162_rn(0.03125f),
                                             one = __float2bfloat162_rn(1.0f);
                        if (b < q4) {                    // a batch left of the diagonal is seen whole
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const __nv_bfloat162 s2 = __floats2bfloat162_rn(__uint_as_float(sc[2 * i]), __uint_as_float(sc[2 * i + 1]));
                                const __nv_bfloat162 w2 = __hfma2(s2, __hfma2(s2, c2, c1), one);
                                pk[i] = *reinterpret_cast<const uint32_t*>(&w2);
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const __nv_bfloat162 s2 = __floats2bfloat162_rn(__uint_as_float(sc[2 * i]), __uint_as_float(sc[2 * i + 1]));
                                const __nv_bfloat162 w2 = __hfma2(s2, __hfma2(s2, c2, c1), one);
                                pk[i] = *reinterpret_cast<const uint32_t*>(&w2) & dm[i];
                            }
                        }
                    } else {
                        // fp32 polynomial on pairs of scores (two-wide fp32 multiply-add): t = s/32 + 1/4, w = s t + 1
                        const uint64_t k2 = f32x2(__float_as_uint(0.03125f), __float_as_uint(0.03125f)),
                                       k1 = f32x2(__float_as_uint(0.25f), __float_as_uint(0.25f)),
                                       k0 = f32x2(__float_as_uint(1.0f), __float_as_uint(1.0f));
                        uint64_t den2 = f32x2(__float_as_uint(den0), __float_as_uint(den1));
                        if (b < q4) {                    // fully visible batch: no mask
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const uint64_t s2 = f32x2(sc[2 * i], sc[2 * i + 1]);
                                const uint64_t w2 = fma2(s2, fma2(s2, k2, k1), k0);
                                den2 = add2(den2, w2);
                                float w0, w1;
                                f32x2_split(w2, w0, w1);
                                pk[i] = pack_bf16(w0, w1);
                            }
                            f32x2_split(den2, den0, den1);
                        } else {                         // the batch that holds the diagonal
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const uint64_t s2 = f32x2(sc[2 * i], sc[2 * i + 1]);
                                float w0, w1;
                                f32x2_split(fma2(s2, fma2(s2, k2, k1), k0), w0, w1);
                                w0 = (2 * i <= lane) ? w0 : 0.f;
                                w1 = (2 * i + 1 <= lane) ? w1 : 0.f;
                                den0 += w0;
                                den1 += w1;
                                pk[i] = pack_bf16(w0, w1);
                            }
                        }
                    }
                }
                if (PQT && b == 3) {               // every score column has been read: phi(Q) may take the upper half
                    tc_fence_before();
                    mbar_arrive(&bars[kTR + t_idx(c)]);
                }
                if (b <= q4) tmem_st16(tmem_addr(tb, lane_base, colTc + b * 16), pk);
                else tmem_st16(tmem_addr(tb, lane_base, colTc + b * 16), zz);
            }
            if constexpr (!PKW) s_den[(c & 3) * kC + tid] = den0 + den1;
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&bars[kP + t_idx(c)]);
            if (tid == 96) TRACE(2, c, 1);
        }
    }

    // ---- final state: into the workspace slot (state pass) or, folded back into the caller's layout, into the
    // caller's state (a piece that ends its head).  Every thread of the first sixteen warps owns a lane of S^T (its
    // warp's lane quarter), so the four role groups share the ten 16-column blocks: the write is 140 KB per head at
    // d_v 128, a fifth of a chunk's time when one group does it alone.
    if (warp < 16) {
        const bool write_ws = STATE_ONLY;
        const bool write_abi = !STATE_ONLY && p.kv_abi != nullptr && head_end;
        if (write_ws || write_abi) {
            const int part = warp >> 2;                                  // 0 row, 1 feature, 2 state, 3 output group
            const int t = ((warp & 3) << 5) + lane;
            const int srow = (t < C::kSLanes) ? t : -1;
            const bool is_z = (DV == 64) && t == 64;
            const int z1f = (DV == 128 && (t & 31) < 16 && (t >> 5) < 2) ? 128 + (t >> 5) * 16 + (t & 15) : -1;
            const int dv = p.dv;
            // without chunks there is no last MMA to wait for, and only the state group knows the state is initialised
            const bool shared = ntot > 0;
            if (ok && shared) ok = mbar_wait(&bars[kFin], 0, abort_flag);
            tc_fence_after();
            if (ok && (shared || part == 2)) {
                float* wseg = p.ws + (size_t)(ws_out < 0 ? 0 : ws_out) * seg_state_floats(DV);
                float* kvo = write_abi ? p.kv_abi + (size_t)head * abi_nrows * dv : nullptr;
                float* zo = write_abi ? p.z_abi + (size_t)head * abi_nrows : nullptr;
                auto put = [&](int f, float v, bool zrow, int col) {
                    if (write_ws) {
                        if (zrow) wseg[(size_t)kF * DV + f] = v;
                        else wseg[(size_t)f * DV + col] = v;
                        return;
                    }
                    const short2 ar = s_abi[f];
                    if (ar.x < 0) return;
                    if (ar.y >= 0) v *= kRsqrt2;
                    if (zrow) { zo[ar.x] = v; if (ar.y >= 0) zo[ar.y] = v; }
                    else if (col < dv) { kvo[(size_t)ar.x * dv + col] = v; if (ar.y >= 0) kvo[(size_t)ar.y * dv + col] = v; }
                };
#pragma unroll 1
                for (int b = shared ? part : 0; b < kF / 16; b += shared ? 4 : 1) {
                    uint32_t r[16];
                    tmem_ld16(tmem_addr(tb, lane_base, C::colS + b * 16), r);
                    tmem_wait_ld();
                    if (srow >= 0) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) put(b * 16 + i, __uint_as_float(r[i]), is_z, srow);
                    }
                }
                if (DV == 128 && part == 2) {
                    uint32_t z0, z1;
                    tmem_ld1(tmem_addr(tb, lane_base, C::colZ0), z0);
                    tmem_ld1(tmem_addr(tb, lane_base, C::colZ1), z1);
                    tmem_wait_ld();
                    put(t, __uint_as_float(z0), true, 0);
                    if (z1f >= 0) put(z1f, __uint_as_float(z1), true, 0);
                }
            }
        }
    }

    if (!ok && lane == 0) atomicOr(p.err, 1u);
    // ---- teardown: everyone meets; after a give-up, loads still in flight get time to land
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int it = 0; it < 200; ++it) __nanosleep(1000);   // ~0.2 ms: far longer than any TMA load in flight
    }
    __syncthreads();
    if (warp == kWarpMma) tmem_dealloc(tb, 512);
    if (tid == 0) { TRACE(5, 1, 7); TRACE_CTA(1); }     // kernel exit
}

// --------------------------------------------------------------------------------- host side
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
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

// [BH][L][width] bf16, box = [1][128][box_w]
bool make_map(CUtensorMap* m, const void* base, int BH, int L, int width, int box_w, CUtensorMapSwizzle sw) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)width, (cuuint64_t)L, (cuuint64_t)BH};
    cuuint64_t strides[2] = {(cuuint64_t)width * 2, (cuuint64_t)L * width * 2};
    cuuint32_t box[3] = {(cuuint32_t)box_w, (cuuint32_t)kC, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

#ifdef BASED_TRACE
unsigned long long* g_trace = nullptr;
#endif

// A launch with programmatic stream serialization: the grid's CTAs may be scheduled before the grid ahead of it in
// the stream has completed, namely once every CTA of that grid has signalled (griddepcontrol.launch_dependents) or
// left; what they may touch before that grid is complete is the kernel's business (griddepcontrol.wait).  Behind a
// kernel that never signals, such a launch behaves like a plain one.  Two uses.  The main pass behind a state pass
// of the same call: every CTA of the state pass signals at its start, so the main pass's CTAs start as SMs come free
// (they cannot take an SM that a CTA of the state pass still needs, all of those being resident or done by then),
// and the one group that reads what the state pass wrote waits for its completion.  The recompute-mode kernel behind
// whatever precedes the call: it waits right after its set-up.
template <int DV, int MODE>
cudaError_t launch_dependent(dim3 grid, cudaStream_t stream, const CUtensorMap& tq, const CUtensorMap& tk,
                             const CUtensorMap& tv, const CUtensorMap& to, const Params& p) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = Cfg<DV>::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, prefill_tc_kernel<DV, MODE>, tq, tk, tv, to, p);
}

// The caller's state of a continued call, folded into the internal basis, as the first workspace slot of each head
// (slot layout: [160 features][DV] values, then the 160 K-state entries).  With a state pass the segments of a head
// take it like the state of an earlier segment and never read the caller's arrays, which the head's last segment
// overwrites with the final state at its end: a segment that started late (the call's CTAs are scheduled as SMs come
// free) could otherwise read what a short last segment had already written.
template <int DV>
__global__ void __launch_bounds__(DV) abi_to_slot_kernel(const float* __restrict__ kv, const float* __restrict__ z,
                                                          float* __restrict__ ws, int per_head, int dv, int sym) {
    const int head = blockIdx.y, f = blockIdx.x, col = threadIdx.x;
    const AbiRows ar = sym ? sym_rows(f) : abi_rows(f);
    const int nrows = sym ? kDSym : kD;
    float* slot = ws + (size_t)head * per_head * seg_state_floats(DV);
    const float* kvh = kv + (size_t)head * nrows * dv;
    float val = 0.f;
    if (ar.a >= 0 && col < dv) val = ar.b >= 0 ? (kvh[(size_t)ar.a * dv + col] + kvh[(size_t)ar.b * dv + col]) * kRsqrt2 : kvh[(size_t)ar.a * dv + col];
    slot[(size_t)f * DV + col] = val;
    if (col == 0) {
        const float* zh = z + (size_t)head * nrows;
        slot[(size_t)kF * DV + f] = ar.a < 0 ? 0.f : (ar.b >= 0 ? (zh[ar.a] + zh[ar.b]) * kRsqrt2 : zh[ar.a]);
    }
}

// Running sum over each head's partial states, in place, between the state pass and the main pass: afterwards a
// head's slot i holds the state of everything in the head up to the end of piece i, so a piece of the main pass
// starts from one slot.  (Summing the earlier pieces' slots in the main pass itself cost its state group 2.7 us of
// load latency per slot before the first state update could run: 11 us on cfg 5's last pieces, 46 us with 18 pieces
// per head.)  per_head > 0: head h owns slots h per_head .. (h + 1) per_head - 1; otherwise the equal chunk
// ranges of prefill_tc_kernel (n ranges, nchr chunks per head, pad w): head h owns the slots of the ranges from
// the one with its first chunk to the one before the range with its last chunk.
__global__ void __launch_bounds__(256) slot_scan_kernel(float* __restrict__ ws, uint32_t floats, int per_head, uint32_t heads,
                                                        uint32_t n, uint32_t nchr, uint32_t w) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");      // the main pass may be scheduled behind this grid
    asm volatile("griddepcontrol.wait;" ::: "memory");                   // the state pass is complete
    const uint32_t h = blockIdx.y;
    uint32_t first, count;
    if (per_head > 0) {
        first = h * (uint32_t)per_head;
        count = (uint32_t)per_head;
    } else {
        const uint32_t nchh = nchr + w, T = heads * nchh;
        auto range_of = [&](uint32_t x) -> uint32_t { return ((x + 1) * n + T - 1) / T - 1; };
        first = range_of(h * nchh + w);
        count = range_of((h + 1) * nchh - 1) - first;
    }
    // one element per thread, eight slots' loads in flight at a time
    const uint32_t e = blockIdx.x * 256 + threadIdx.x;
    if (e >= floats) return;
    float* col = ws + (size_t)first * floats + e;
    float acc = 0.f;
#pragma unroll 1
    for (uint32_t i = 0; i < count; i += 8) {
        float v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = (i + j < count) ? col[(size_t)(i + j) * floats] : 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            acc += v[j];
            if (i + j < count) col[(size_t)(i + j) * floats] = acc;
        }
    }
}

static cudaError_t launch_slot_scan(float* ws, int dv_kernel, int per_head, int heads, int n, int nchr, int w, cudaStream_t stream) {
    const uint32_t floats = (uint32_t)seg_state_floats(dv_kernel);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((floats + 255) / 256, heads);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, slot_scan_kernel, ws, floats, per_head, (uint32_t)heads, (uint32_t)n, (uint32_t)nchr, (uint32_t)w);
}

template <int DV>
based_status launch_dv(const void* q, const void* k, const void* v, void* out, float* kv, float* z, int BH, int L,
                       int dv, int flags, float* ws, const SegPlan plan, cudaStream_t stream) {
    using C = Cfg<DV>;
    CUtensorMap tq, tk, tv, to;
    if (!make_map(&tq, q, BH, L, kDFeat, kDFeat, CU_TENSOR_MAP_SWIZZLE_32B) ||
        !make_map(&tk, k, BH, L, kDFeat, kDFeat, CU_TENSOR_MAP_SWIZZLE_32B) ||
        !make_map(&tv, v, BH, L, dv, 64, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map(&to, out, BH, L, dv, 64, CU_TENSOR_MAP_SWIZZLE_128B))
        return BASED_ERR_CUDA;
    Params p{};         // (every field the kernel may read has a value: pad is read on every path)
    p.kv_abi = kv;
    p.z_abi = z;
    p.ws = ws;
    if (error_word_ptr(&p.err) != BASED_OK) return BASED_ERR_CUDA;
    p.L = L;
    const int nseg = plan.nseg;
    const bool recompute = plan.recompute;
    p.nseg = nseg;
    p.seg_len = plan.per * kC;
    p.continue_abi = (flags & BASED_STATE_CONTINUE) ? 1 : 0;
    p.sym = (flags & BASED_STATE_SYM) ? 1 : 0;
    p.numerator_only = (flags & BASED_NUMERATOR_ONLY) ? 1 : 0;
    p.dv = dv;
#ifdef BASED_TRACE
    p.trace = g_trace;
#endif
    {
        static bool configured[64] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BASED_ERR_CUDA;
        std::lock_guard<std::mutex> lock(setup_mutex());
        if (!configured[dev]) {
            if (cudaFuncSetAttribute(prefill_tc_kernel<DV, kModeMain>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)C::kSmemBytes) != cudaSuccess ||
                cudaFuncSetAttribute(prefill_tc_kernel<DV, kModeState>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)C::kSmemBytes) != cudaSuccess ||
                cudaFuncSetAttribute(prefill_tc_kernel<DV, kModePre>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)C::kSmemBytes) != cudaSuccess)
                return BASED_ERR_CUDA;
            configured[dev] = true;
        }
    }
    p.balanced = 0;
    p.heads = BH;
    if (plan.balanced > 0) {
        // state pass over every piece that ends inside its head, (d_v 64) the running sums of each head's slots, then
        // the main pass; both passes on one row of CTAs: one per range, then one per head boundary
        p.balanced = plan.balanced;
        p.nseg = 1;
#ifdef BASED_PAD
        p.pad = BASED_PAD;
#else
        p.pad = 5;
#endif
        const dim3 grid(plan.balanced + BH - 1, 1);
        prefill_tc_kernel<DV, kModeState><<<grid, kThreads, C::kSmemBytes, stream>>>(tq, tk, tv, to, p);
        note_launch();
        based_status st = check_launch("prefill_tc_kernel<state, balanced>");
        if (st != BASED_OK) return st;
        if (C::kSlotScan) {
            if (launch_slot_scan(ws, DV, 0, BH, plan.balanced, (L + kC - 1) / kC, p.pad, stream) != cudaSuccess) return BASED_ERR_CUDA;
            note_launch();
            st = check_launch("slot_scan_kernel");
            if (st != BASED_OK) return st;
        }
        if (launch_dependent<DV, kModeMain>(grid, stream, tq, tk, tv, to, p) != cudaSuccess) return BASED_ERR_CUDA;
        note_launch();
        return check_launch("prefill_tc_kernel<balanced>");
    }
    if (nseg > 1 && recompute) {
        if (launch_dependent<DV, kModePre>(dim3(nseg, BH), stream, tq, tk, tv, to, p) != cudaSuccess) return BASED_ERR_CUDA;
        note_launch();
        return check_launch("prefill_tc_kernel<pre>");
    }
    if (nseg > 1) {
        based_status st;
        if (p.continue_abi) {
            // the caller's state goes into each head's first slot (see abi_to_slot_kernel); no segment reads it itself
            p.pad = 1;
            p.continue_abi = 0;
            abi_to_slot_kernel<DV><<<dim3(kF, BH), DV, 0, stream>>>(kv, z, ws, nseg, dv, p.sym);
            note_launch();
            st = check_launch("abi_to_slot_kernel");
            if (st != BASED_OK) return st;
        }
        prefill_tc_kernel<DV, kModeState><<<dim3(nseg - 1, BH), kThreads, C::kSmemBytes, stream>>>(tq, tk, tv, to, p);
        note_launch();
        st = check_launch("prefill_tc_kernel<state>");
        if (st != BASED_OK) return st;
        if (C::kSlotScan && nseg - 1 + p.pad > 1) {     // (one slot per head is its own running sum)
            if (launch_slot_scan(ws, DV, nseg - 1 + p.pad, BH, 0, 0, 0, stream) != cudaSuccess) return BASED_ERR_CUDA;
            note_launch();
            st = check_launch("slot_scan_kernel");
            if (st != BASED_OK) return st;
        }
    }
    if (nseg > 1) {
        if (launch_dependent<DV, kModeMain>(dim3(nseg, BH), stream, tq, tk, tv, to, p) != cudaSuccess) return BASED_ERR_CUDA;
    } else {
        prefill_tc_kernel<DV, kModeMain><<<dim3(nseg, BH), kThreads, C::kSmemBytes, stream>>>(tq, tk, tv, to, p);
    }
    note_launch();
    return check_launch("prefill_tc_kernel");
}

}  // namespace

// How a head's sequence is cut into segments so that about one CTA per SM is busy.
//  - one segment: the plain chunk loop;
//  - state pass: a first launch computes every segment's own state into the workspace, the main
//    launch starts each segment from the sum of the earlier ones (long sequences; d_v 64: a small kernel in
//    between turns the partial states into running sums, see Cfg::kSlotScan);
//  - recompute: one launch, no workspace; a segment's CTA first runs the state update alone over
//    all earlier chunks (short sequences, where a second launch and start-up cost more than that).
// The choice compares modelled CTA times in thousands of cycles, constants fitted on B200 with every SM busy:
// full chunk 3.0 (d_v 64) / 4.1 (d_v 128), state-update-only chunk of the state pass 1.1 / 2.2, of the recompute
// mode 1.5 / 2.6, a state pass ahead of the main pass 34 / 30 (its CTAs' start-up and tail, the slot sums, the
// launches).  In recompute mode later segments do more redundant work, so the first n - 1 segments get `per`
// chunks each and the last one the (shorter) rest, `per` chosen to level the modelled times.  (Forced plans
// against this choice on 23 shapes between 1 and 128 heads that do not take the equal chunk ranges: within 4 % of the
// best forced plan on every one.)
// ws_limit: bytes of workspace the plan may use (plans that need more are not considered).
static SegPlan prefill_tc_plan(int BH, int L, int d_v, bool continued = false, size_t ws_limit = ~(size_t)0) {
    const int nch = (L + kC - 1) / kC;
    const size_t slot = seg_state_floats(d_v) * sizeof(float);
    const float full = d_v == 64 ? 3.0f : 4.1f, upd = d_v == 64 ? 1.1f : 2.2f;
    const float second = d_v == 64 ? 34.f : 30.f;   // a state pass ahead of the main pass: its own start-up and tail, the slot sums, the launches
    // a pre-chunk of the recompute mode costs more than a chunk of the state pass (its kernel keeps four stages of
    // q + k + v size and the whole chunk loop's code); d_v 64: of 1.0 / 1.5 / 2.0 / 2.4 this value gave the shortest
    // cfg-2 calls; d_v 128: the smallest value that keeps B1 H8 L4096 on four state-pass segments (35.5 against 43 us)
    const float pre = d_v == 64 ? 1.5f : 2.6f;
    int nmax = 148 / BH;
    if (nmax > 8) nmax = 8;
    // state pass: as many segments as SMs allow (at least two chunks each); its fixed cost decides against short ones
    int nseg = nmax;
    if (nseg > nch / 2) nseg = nch / 2;
    if (nseg < 1) nseg = 1;
    while (nseg > 1 && ((nch + nseg - 1) / nseg) * (nseg - 1) >= nch) --nseg;   // every segment owns a chunk
    while (nseg > 1 && ((size_t)BH * (nseg - 1 + (continued ? 1 : 0)) * slot > ws_limit ||       // (a continued call: + the caller's state)
                        ((nch + nseg - 1) / nseg) * (nseg - 1) >= nch))
        --nseg;
    SegPlan best = {nseg, (nch + nseg - 1) / nseg, false, 0};
    float best_cost = nseg > 1 ? (float)best.per * (upd + full) + second : (float)nch * full;
    for (int n = 2; n <= nmax; ++n) {
        for (int per = (nch + n - 1) / n; per * (n - 1) < nch; ++per) {
            float cost = 0.f;
            for (int j = 0; j < n; ++j) {
                const int own = (j == n - 1) ? nch - per * (n - 1) : per;
                const float c = (float)(j * per) * pre + (float)own * full;
                if (c > cost) cost = c;
            }
            // (between recompute plans of equal modelled cost the one with more segments keeps more SMs busy)
            if (cost < 0.95f * best_cost || (best.recompute && n > best.nseg && cost <= best_cost)) {
                best = {n, per, true, 0};
                best_cost = cost;
            }
        }
    }
    //  - balanced: all heads' chunks, laid end to end, are cut into 148 equal ranges, one per SM (a range then
    //    holds the tail of one head and the start of the next, run as two CTAs on the same SM one after the
    //    other); state pass and main pass as above.  It fills every SM whatever the head count.  Not for
    //    continued calls: a head's last piece writes the caller's state while the first piece of the same head,
    //    queued behind another head's tail, may not have read it yet.
    if (BH < 148 && !continued) {
        const long long total = (long long)BH * nch;
        const int ranges = 148;
        const float share = (float)((total + ranges - 1) / ranges);
        const float cost = share * (upd + full) + second + 7.f;      // a second CTA's start-up on some SMs
        if (share >= 16.f && total >= ranges && total <= 14000000 && (size_t)ranges * slot <= ws_limit && cost < 0.95f * best_cost)
            best = {1, nch, false, ranges};
    }
#ifdef BASED_TRACE
    if (const char* e = getenv("BASED_NSEG")) {
        const int v = atoi(e);                      // negative: recompute mode with that many segments
        best.nseg = v < 0 ? -v : (v > 0 ? v : 1);
        best.recompute = v < 0;
        best.per = (nch + best.nseg - 1) / best.nseg;
        if (const char* q = getenv("BASED_PER")) best.per = atoi(q);
    }
#endif
    return best;
}

// ---- the state of a token block without its outputs ---------------------------------------------
// Segments of the state-update-only pass for a state-only call: up to eight per head, about one CTA per SM.
static SegPlan prefill_tc_state_plan(int BH, int L) {
    const int nch = (L + kC - 1) / kC;
    int n = 148 / BH;
    n = n < 1 ? 1 : (n > 8 ? 8 : n);
    if (n > nch) n = nch;
    const int per = (nch + n - 1) / n;
    return {(nch + per - 1) / per, per, false, 0};
}

// Sum of a head's partial states (internal basis, [160][DV] + [160] per segment) into the caller's state
// (273 rows, or the 153 symmetric ones), added to it when `cont`.
template <int DV>
__global__ void __launch_bounds__(256) state_reduce_kernel(const float* __restrict__ ws, int nseg, float* __restrict__ kv,
                                                           float* __restrict__ z, int dv, int sym, int cont) {
    const size_t head = blockIdx.x;
    const size_t stride = seg_state_floats(DV);
    const float* wh = ws + head * nseg * stride;
    const int nrows = sym ? kDSym : kD;
    float* kvh = kv + head * (size_t)nrows * dv;
    float* zh = z + head * (size_t)nrows;
    // blockIdx.y: a block of 8 internal features (their DV value columns and their K-state entries)
    const int f0 = blockIdx.y * 8;
    for (int e = threadIdx.x; e < 8 * (DV + 1); e += 256) {
        const bool zrow = e >= 8 * DV;
        const int f = f0 + (zrow ? e - 8 * DV : e / DV), col = zrow ? 0 : e % DV;
        const int idx = zrow ? kF * DV + f : f * DV + col;
        const AbiRows ar = sym ? sym_rows(f) : abi_rows(f);
        if (ar.a < 0 || (!zrow && col >= dv)) continue;
        float acc = 0.f;
        for (int sg = 0; sg < nseg; ++sg) acc += wh[sg * stride + idx];
        if (ar.b >= 0) acc *= kRsqrt2;
        float* dst = zrow ? zh : kvh + col;
        const size_t pitch = zrow ? 1 : (size_t)dv;
        dst[ar.a * pitch] = acc + (cont ? dst[ar.a * pitch] : 0.f);
        if (ar.b >= 0) dst[ar.b * pitch] = acc + (cont ? dst[ar.b * pitch] : 0.f);
    }
}

template <int DV>
static based_status launch_state_dv(const void* k, const void* v, float* kv, float* z, int BH, int L, int dv, int flags,
                                    float* ws, cudaStream_t stream) {
    using C = Cfg<DV>;
    const SegPlan plan = prefill_tc_state_plan(BH, L);
    CUtensorMap tk, tv;
    if (!make_map(&tk, k, BH, L, kDFeat, kDFeat, CU_TENSOR_MAP_SWIZZLE_32B) ||
        !make_map(&tv, v, BH, L, dv, 64, CU_TENSOR_MAP_SWIZZLE_128B))
        return BASED_ERR_CUDA;
    Params p{};
    p.ws = ws;
    if (error_word_ptr(&p.err) != BASED_OK) return BASED_ERR_CUDA;
    p.L = L;
    p.nseg = plan.nseg + 1;            // the workspace holds nseg - 1 partial states per head
    p.heads = BH;
    p.seg_len = plan.per * kC;
    p.dv = dv;
#ifdef BASED_TRACE
    p.trace = g_trace;
#endif
    {
        static bool configured[64] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BASED_ERR_CUDA;
        std::lock_guard<std::mutex> lock(setup_mutex());
        if (!configured[dev]) {
            if (cudaFuncSetAttribute(prefill_tc_kernel<DV, kModeState>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)C::kSmemBytes) != cudaSuccess)
                return BASED_ERR_CUDA;
            configured[dev] = true;
        }
    }
    // the q and output maps are not used by the state-update-only pass
    prefill_tc_kernel<DV, kModeState><<<dim3(plan.nseg, BH), kThreads, C::kSmemBytes, stream>>>(tk, tk, tv, tv, p);
    note_launch();
    based_status st = check_launch("prefill_tc_kernel<state>");
    if (st != BASED_OK) return st;
    state_reduce_kernel<DV><<<dim3(BH, kF / 8), 256, 0, stream>>>(ws, plan.nseg, kv, z, dv, (flags & BASED_STATE_SYM) ? 1 : 0,
                                                                  (flags & BASED_STATE_CONTINUE) ? 1 : 0);
    note_launch();
    return check_launch("state_reduce_kernel");
}

size_t prefill_tc_state_workspace_bytes(int BH, int L, int d_v) {
    if (d_v == 112) d_v = 128;
    return (size_t)BH * prefill_tc_state_plan(BH, L).nseg * seg_state_floats(d_v) * sizeof(float);
}

based_status launch_prefill_tc_state(const void* k, const void* v, float* kv, float* z, int BH, int L, int d_v,
                                     int flags, void* workspace, cudaStream_t stream) {
    float* ws = static_cast<float*>(workspace);
    if (d_v == 64) return launch_state_dv<64>(k, v, kv, z, BH, L, 64, flags, ws, stream);
    return launch_state_dv<128>(k, v, kv, z, BH, L, d_v, flags, ws, stream);      // 112 or 128
}

size_t prefill_tc_workspace_bytes(int BH, int L, int d_v) {
    if (d_v == 112) d_v = 128;                      // runs on the d_v 128 kernel, partial states in its layout
    // the larger of the two plans a call can take (continued calls do not use the balanced one)
    size_t need = 0;
    for (int cont = 0; cont < 2; ++cont) {
        const SegPlan plan = prefill_tc_plan(BH, L, d_v, cont != 0);
        size_t n = 0;
        if (plan.balanced > 0) n = (size_t)plan.balanced * seg_state_floats(d_v) * sizeof(float);
        else if (!plan.recompute && plan.nseg > 1) n = (size_t)BH * (plan.nseg - 1 + cont) * seg_state_floats(d_v) * sizeof(float);
        need = n > need ? n : need;
    }
    return need;
}

based_status launch_prefill_tc(const void* q, const void* k, const void* v, void* out, float* kv, float* z, int BH,
                               int L, int d_v, int flags, void* workspace, cudaStream_t stream, size_t workspace_limit) {
    const SegPlan plan = prefill_tc_plan(BH, L, d_v == 112 ? 128 : d_v, (flags & BASED_STATE_CONTINUE) != 0,
                                         workspace ? workspace_limit : 0);
    float* ws = static_cast<float*>(workspace);
    if (d_v == 64) return launch_dv<64>(q, k, v, out, kv, z, BH, L, 64, flags, ws, plan, stream);
    return launch_dv<128>(q, k, v, out, kv, z, BH, L, d_v, flags, ws, plan, stream);      // 112 or 128
}

}  // namespace based

#ifdef BASED_TRACE
// out[0..127]: the per-warp wait records; out[128]: owner CTA; then both are cleared
extern "C" void based_debug_read_waits(unsigned int* out) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(out, based::sm100::g_wait_dbg, sizeof(unsigned int) * 128);
    cudaMemcpyFromSymbol(out + 128, based::sm100::g_wait_owner, sizeof(unsigned int));
    unsigned int zero[129] = {};
    cudaMemcpyToSymbol(based::sm100::g_wait_dbg, zero, sizeof(unsigned int) * 128);
    cudaMemcpyToSymbol(based::sm100::g_wait_owner, zero, sizeof(unsigned int));
}
extern "C" void based_debug_set_trace(void* ptr) { based::g_trace = static_cast<unsigned long long*>(ptr); }
#endif
