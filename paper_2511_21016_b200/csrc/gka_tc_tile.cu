// tcgen05 / TMEM chunk-wise GKA forward (bf16 operands, fp32 accumulation) for sm_100a, token-major tiles.
//
// One persistent thread block per SM walks its range of chunks (gka_common.cuh explains the work
// decomposition) in tiles of up to two chunks = 128 tokens.  A tile puts one token on each TMEM lane, so
// every product of the chunk-wise form (Section 4.2.1; Algorithm 1 on the whole tile) is an M = 128 tile:
//     S[c][j]  = sum_e X'[c][e] K[j][e]                        scores      (A = X', B = K, both K-major)
//     P[c][j]  = S[c][j] * Gamma[c][j] / zt_c  for j <= c        masked, as packed bf16 back into TMEM
//     Y[c][d]  = sum_e X'[c][e] H_0[d][e] + sum_j P[c][j] Kw[j][d]   (second product: A = P from TMEM)
//     x_c     <- x_c + beta (x_c - x_c^prev) + sigma (q_c - Y_c - lambda_c x_c)          Algorithm 1
//     O[c][i]  = sum_e X'[c][e] U_0[i][e] + sum_j P[c][j] V[j][i]
// with X' = zt_c x_c in bf16, zt_c = max(zeta_c, 2^-60).  16 compute warps: warp quadrant q owns tokens
// 32 q .. 32 q + 31 (its TMEM lanes), column quarter cq owns 32 of the 128 columns; a thread therefore
// holds one token's 32 channels of x, x - x^prev and q in registers, and every per-token coefficient of
// Algorithm 1 (sigma_c, beta_c, lambda_c, zt_c) is a per-thread scalar.
//
// Decay factors.  Gamma[c][j] / zt_c = 2^(G_c - G_j) / zt_c (G the cumulative log2 gate in the tile).  When
// the whole tile decays by less than 2^-60 this is 2^-G_last * w_j with w_j = 2^(G_last - G_j) <= 1, the
// weight the state update needs anyway: the B operand of the second product is Kw = w o K and P needs one
// tile-wide constant factor.  Tiles that decay more (and the last score pass, whose P multiplies the
// unweighted V) compute the factor per element and pair P with the unweighted operand.
//
// State: fp32 masters of H and U live in TMEM (2 x 128 columns) for a whole run; per tile each is read once
// (bf16 operand copy to shared memory, ||H_0||_F^2), scaled by the tile's decay and advanced by tensor-core
// products K^T Kw, V^T Kw.  The Frobenius norms of Section 4.2.1 come from K H_0 and the Gram matrix K K^T
// (two more tensor-core products per tile) and an affine scan over the tile's tokens.
//
// One thread of an extra warpgroup (kept at 32 registers by setmaxnreg) issues every tcgen05.mma; the
// compute warps post requests through an mbarrier and wait for tcgen05.commit.  K tiles are double
// buffered (the next tile's K is fetched by TMA during the solve), V arrives during the solve as well.
#include <cuda.h>

#include "gka_common.cuh"
#include "gka_tc_util.cuh"

namespace gka {
namespace {

using namespace tcu;

constexpr int D = 128;
constexpr int NT = 128;                    // tokens per tile: one per TMEM lane
constexpr int CT = 512;                    // compute threads
constexpr int kThreadsTile = CT + 128;     // + the warpgroup that holds the MMA-issuing thread
constexpr int kRegsCompute = 112, kRegsIssuer = 32;   // register split after setmaxnreg (launch: 96 each)
// setmaxnreg.inc waits, without a bound, for registers that the other warpgroup gives back: the split must fit
// what the block was launched with
static_assert(CT * kRegsCompute + 128 * kRegsIssuer <= kThreadsTile * 96, "register split exceeds the launch allocation");

// ---- shared memory map (bytes; every operand buffer is 1024-byte aligned).  A [128 rows][128 columns] bf16
// operand is two boxes of [128 rows][64 columns] with the 128-byte swizzle, 16384 bytes apart.
constexpr uint32_t OFF_K0 = 0;           // K tile, stage 0 (rows = keys)
constexpr uint32_t OFF_K1 = 32768;       // K tile, stage 1
constexpr uint32_t OFF_V = 65536;        // V tile
constexpr uint32_t OFF_KW = 98304;       // w o K
constexpr uint32_t OFF_H = 131072;       // bf16 H_0 (later U_0), rows = state rows
constexpr uint32_t OFF_X = 163840;       // X' (rows = tokens)
constexpr uint32_t OFF_SC = 196608;      // scalars
// Per-token scalars that depend on the gates and the other per-token inputs alone: a helper warp prepares them
// one tile ahead, into the buffer the tile's parity selects.
struct GateScalars {
    float lg[NT];          // log2 gamma_c
    float G2[NT];          // cumulative log2 gate
    float ac[NT];          // G2_c - max(G2_c, -60): exponent correction of clamped tokens
    float zt[NT];          // clamped zeta_c
    float lam[NT];         // lambda_c as given
    float al[NT];          // alpha_c of the tile's tokens (alpha-connection)
    float sb[NT];          // sqrt(beta_j) of the tile's keys (beta-augmented write)
    __align__(16) float iz[NT];   // 2^-G2_c (tiles that are not clamped)
};
struct TileScalars {
    GateScalars g[2];
    float G2cur[NT];       // copy of the current tile's cumulative log2 gates at a fixed place (read inside the solve loop)
    float lam[NT];         // lambda_c (after the adaptive rule, if any)
    float s0[NT];          // 2 / (L + mu)
    float rho2[NT];
    float part[2][4][NT];  // Frobenius partial sums: [k H_0 k | Gram part][column quarter][key]
    float carry[2][2][4];  // per-warp totals (a, b) of the two scans
    float red[16];         // per-warp sums of squares of H_0
    int req_op;            // request to the MMA issuer
    int stop;              // block-wide copy of the abort flag, taken between tiles
};
constexpr uint32_t SC_BYTES = 15360;
static_assert(sizeof(TileScalars) <= SC_BYTES, "scalar block too large");
constexpr uint32_t TILE_SMEM = OFF_SC + SC_BYTES + 1024;   // + slack for the 1024-byte alignment of the base

// ---- TMEM columns: fp32 masters H, U; score accumulator S (P overwrites it in place); Y / O accumulator
constexpr uint32_t TM_H = 0, TM_U = 128, TM_S = 256, TM_Y = 384;

enum { BAR_K0 = 0, BAR_K1, BAR_V, BAR_A, BAR_B, BAR_G0, BAR_G1, BAR_COUNT };   // G: gate scalars of a buffer are ready
enum { OP_FROB = 1, OP_ITER1, OP_ITER1_LAST, OP_ITER2, OP_OUT, OP_EXIT, OP_GRAM, OP_NONE, OP_OUT_U0 };
constexpr int OPF_STAGE = 1 << 8, OPF_PLAIN_K = 1 << 9;   // request flags: K stage; pair P with K instead of w o K

// ---- operand descriptor constants relative to (shared base >> 4); k-steps of 16
__host__ __device__ constexpr uint32_t t_kmaj(uint32_t off) { return (off >> 4) | ((16u >> 4) << 16); }
__host__ __device__ constexpr uint32_t t_mn(uint32_t off) { return (off >> 4) | ((16384u >> 4) << 16); }
__host__ __device__ constexpr uint32_t t_kstep(int ks) { return (uint32_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4); }
__host__ __device__ constexpr uint32_t t_mnstep(int ks) { return (uint32_t)((ks * 2048) >> 4); }

// D (+)= A x B, both operands in shared memory: low words are a base register plus an immediate
template <int ACC, uint32_t A_CONST, uint32_t B_CONST>
__device__ __forceinline__ void mma_ss2(uint32_t d_tmem, uint32_t a_base, uint32_t b_base, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .b64 da, db;\n\t.reg .b32 la, lb;\n\t"
        "add.u32 la, %1, %5;\n\tadd.u32 lb, %2, %6;\n\t"
        "mov.b64 da, {la, %4};\n\tmov.b64 db, {lb, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, %7;\n\t}" ::"r"(d_tmem), "r"(a_base), "r"(b_base), "r"(idesc),
        "r"(kDescHi), "n"(A_CONST), "n"(B_CONST), "n"(ACC)
        : "memory");
}
// D += A x B with A (packed bf16 pairs) in TMEM
template <uint32_t B_CONST>
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_base, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .b64 db;\n\t.reg .b32 lb;\n\t.reg .pred p;\n\t"
        "add.u32 lb, %2, %5;\n\tmov.b64 db, {lb, %4};\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, p;\n\t}" ::"r"(d_tmem), "r"(a_tmem), "r"(b_base), "r"(idesc),
        "r"(kDescHi), "n"(B_CONST)
        : "memory");
}
template <int ACC0, uint32_t A, uint32_t B, int KS = 0>   // both K-major, 8 k-steps over the 128 channels
__device__ __forceinline__ void mma8_kk(uint32_t d, uint32_t a_base, uint32_t b_base, uint32_t idesc) {
    if constexpr (KS < 8) {
        mma_ss2<(KS == 0 ? ACC0 : 1), A + t_kstep(KS), B + t_kstep(KS)>(d, a_base, b_base, idesc);
        mma8_kk<ACC0, A, B, KS + 1>(d, a_base, b_base, idesc);
    }
}
template <uint32_t A, uint32_t B, int KS = 0>   // both MN-major, 8 k-steps over the 128 tokens, accumulating
__device__ __forceinline__ void mma8_mm(uint32_t d, uint32_t a_base, uint32_t b_base, uint32_t idesc) {
    if constexpr (KS < 8) {
        mma_ss2<1, A + t_mnstep(KS), B + t_mnstep(KS)>(d, a_base, b_base, idesc);
        mma8_mm<A, B, KS + 1>(d, a_base, b_base, idesc);
    }
}
template <uint32_t B, int KS = 0>   // A = P in TMEM (a thread's 16 packed columns per column quarter), B MN-major
__device__ __forceinline__ void mma8_pm(uint32_t d, uint32_t p_tmem, uint32_t b_base, uint32_t idesc) {
    if constexpr (KS < 8) {
        mma_ts<B + t_mnstep(KS)>(d, p_tmem + 32 * (KS >> 1) + 8 * (KS & 1), b_base, idesc);
        mma8_pm<B, KS + 1>(d, p_tmem, b_base, idesc);
    }
}

__device__ __forceinline__ void issuer_run(int req, uint32_t base14, uint32_t tmem, uint32_t bars) {
    constexpr uint32_t I_KK = make_idesc(128, 128, 0, 0);   // both operands K-major
    constexpr uint32_t I_PM = make_idesc(128, 128, 0, 1);   // A from TMEM, B MN-major
    constexpr uint32_t I_MM = make_idesc(128, 128, 1, 1);   // both MN-major
    constexpr uint32_t K_k = t_kmaj(0), K_mn = t_mn(0);     // relative to the K stage
    constexpr uint32_t V_mn = t_mn(OFF_V), Kw_mn = t_mn(OFF_KW), H_k = t_kmaj(OFF_H), X_k = t_kmaj(OFF_X);
    const int op = req & 0xFF;
    const uint32_t kb = base14 + ((req & OPF_STAGE) ? (OFF_K1 >> 4) : (OFF_K0 >> 4));
    const uint32_t tm_H = tmem + TM_H, tm_U = tmem + TM_U, tm_S = tmem + TM_S, tm_Y = tmem + TM_Y;
    if (op == OP_ITER1 || op == OP_ITER1_LAST) {
        mma8_kk<0, X_k, K_k>(tm_S, base14, kb, I_KK);
        mma_commit(bars + 8 * BAR_A);
        if (op == OP_ITER1) mma8_kk<0, X_k, H_k>(tm_Y, base14, base14, I_KK);
    } else if (op == OP_ITER2) {
        if (req & OPF_PLAIN_K) mma8_pm<K_mn>(tm_Y, tm_S, kb, I_PM);
        else mma8_pm<Kw_mn>(tm_Y, tm_S, base14, I_PM);
        mma_commit(bars + 8 * BAR_B);
    } else if (op == OP_GRAM) {
        mma8_kk<0, K_k, K_k>(tm_S, kb, kb, I_KK);            // Gram matrix K K^T (completion is covered by OP_FROB's commit)
    } else if (op == OP_FROB) {
        mma8_mm<K_mn, Kw_mn>(tm_H, kb, base14, I_MM);        // H += K^T (w o K)
        mma8_kk<0, K_k, H_k>(tm_Y, kb, base14, I_KK);        // K H_0
        mma_commit(bars + 8 * BAR_A);
    } else if (op == OP_OUT_U0) {
        // X' U_0^T (the H buffer holds U_0 now): posted as soon as U_0 is staged, it runs behind the last score product,
        // under the score epilogue; completion is covered by OP_OUT's first commit
        mma8_kk<0, X_k, H_k>(tm_Y, base14, base14, I_KK);
    } else if (op == OP_OUT) {
        mma8_pm<V_mn>(tm_Y, tm_S, base14, I_PM);             // O = X' U_0^T + P V
        mma_commit(bars + 8 * BAR_A);
        mma8_mm<V_mn, Kw_mn>(tm_U, base14, base14, I_MM);    // U += V^T (w o K)
        mma_commit(bars + 8 * BAR_B);
    }
}

#ifdef GKA_TC_TIMING
// Debug build only: event trace of block 0 (compute thread 0 and the issuing thread).
__device__ long long g_ttrace[2][8192];
__device__ int g_ttrace_n[2];
__shared__ int s_ttrace_n[2];
#define TRACE(role, id)                                                                                        \
    do {                                                                                                       \
        if (blockIdx.x == 0 && s_ttrace_n[role] < 8192)                                                        \
            g_ttrace[role][s_ttrace_n[role]++] = (clock64() << 8) | (long long)(id);                           \
    } while (0)
#if GKA_TC_TIMING == 2   /* light mode: no stamps inside the solve loop, none in waits or in the issuer */
#define TSTAMP(k)                                                         \
    do {                                                                  \
        if (tid == 0 && (k) != 7 && (k) != 8 && (k) != 9 && (k) != 10) TRACE(0, k); \
    } while (0)
#define TRACE_HEAVY(role, id)
#else
#define TSTAMP(k)               \
    do {                        \
        if (tid == 0) TRACE(0, k); \
    } while (0)
#define TRACE_HEAVY(role, id) TRACE(role, id)
#endif
#else
#define TRACE_HEAVY(role, id)
#define TRACE(role, id)
#define TSTAMP(k)
#endif

#define TMEM_ST8(taddr, r)                                                                                       \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(r[0]), \
                 "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])                     \
                 : "memory")

__device__ __forceinline__ void cta_sync() { asm volatile("bar.sync 1, 512;" ::: "memory"); }

// Everything a compute thread needs to know about itself.
struct Ctx {
    int tid, l, q, cq;            // thread, lane in warp, TMEM lane quadrant, column quarter
    int c;                        // token / TMEM lane / state row: 32 q + l
    uint32_t lane_addr;           // (32 q) << 16
    unsigned char *smem;
    TileScalars *sc;
    uint32_t bars, tmem, abort_addr;
};

__device__ __forceinline__ bool aborted(const Ctx &cx) {
    int v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(cx.abort_addr) : "memory");
    return v != 0;
}
// Wait for an mbarrier phase (TMA arrival or tcgen05.commit): every warp polls for itself, bounded; the block
// reports GKA_ERR_TIMEOUT when it ends if a wait gave up.
__device__ __forceinline__ void wait_bar(const Ctx &cx, int which, uint32_t parity) {
    if (!mbar_spin_bounded(cx.bars + 8 * which, parity))
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(cx.abort_addr), "r"(1) : "memory");
#ifdef GKA_TC_TIMING
    if (cx.tid == 0) TRACE_HEAVY(0, 20);
#endif
}
// Block-wide barrier of the compute threads that also hands a batch of MMAs to the issuing warp: the issuer
// sits in the same hardware barrier, so it wakes with the last arriving compute warp.  Every thread's
// writes and fences for the batch come before the call.
__device__ __forceinline__ void sync_post(const Ctx &cx, int req) {
    if (cx.tid == 0) *reinterpret_cast<volatile int *>(&cx.sc->req_op) = req;
    asm volatile("bar.sync 3, 544;" ::: "memory");
}
// byte offset of the 16-byte group holding columns 8 g .. 8 g + 7 (g = 0..15) of row r in a 128 x 128 operand
__device__ __forceinline__ uint32_t tile_off(int r, int g) {
    return (uint32_t)((g >> 3) * 16384 + r * 128 + (((g & 7) ^ (r & 7)) << 4));
}

// One pass over a master (H or U) for this thread's row and 32 columns: source is TMEM, or global memory at
// the start of a run.  Writes the bf16 operand copy, optionally accumulates the sum of squares, scales by the
// tile's decay and stores the result back to TMEM.
// Where a run's start state comes from: the caller's initial state of the sequence (or zero), carried through
// the segment summaries (decay product, delta) of the work items j0 .. j1 - 1 that hold the earlier part of the
// sequence: state <- decay_j * state + delta_j.  `off` selects the master (H or U) and this thread's row.
struct StartSrc {
    const float *state;      // caller's state of the sequence, or nullptr (zero)
    const float *delta;      // summaries [item][st]
    const float *decay;      // [item]
    int j0, j1;
    size_t st, off;
};
// Start of a run: the master's value (this thread's row, 32 columns at `taddr`) is written to TMEM from global
// memory; the regular pass then reads it from there.  Compiled as a function of its own: it runs once per run and
// must not weigh on the register allocation of the per-tile code.  All loads of a step go out together (the
// thread's 128 bytes are one line), so the fold costs one round trip per chain item.
__device__ __noinline__ void master_seed(uint32_t taddr, const float *state, const float *delta, const float *decay,
                                         int j0, int j1, size_t st, size_t e) {
    float g[32];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        // ordinary loads: the start states may come from the scan kernel this kernel overlaps with
        const float4 v4 = state ? *reinterpret_cast<const float4 *>(state + e + 4 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
        g[4 * i + 0] = v4.x; g[4 * i + 1] = v4.y; g[4 * i + 2] = v4.z; g[4 * i + 3] = v4.w;
    }
    for (int j = j0; j < j1; ++j) {
        // summaries come from the kernel this one may overlap with as its programmatic dependent: ordinary loads
        // (visible after the dependency wait), not the read-only path, whose data must not change under the kernel
        const float dj = *reinterpret_cast<const volatile float *>(decay + j);
        float4 dd[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) dd[i] = *(reinterpret_cast<const float4 *>(delta + (size_t)j * st + e) + i);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            g[4 * i + 0] = fmaf(dj, g[4 * i + 0], dd[i].x);
            g[4 * i + 1] = fmaf(dj, g[4 * i + 1], dd[i].y);
            g[4 * i + 2] = fmaf(dj, g[4 * i + 2], dd[i].z);
            g[4 * i + 3] = fmaf(dj, g[4 * i + 3], dd[i].w);
        }
    }
    uint32_t r[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(g[i]);
    TMEM_ST32(taddr, r);
    tmem_wait_st();
}

template <bool SUMSQ>
__device__ __forceinline__ float master_pass(const Ctx &cx, uint32_t tm_master, bool from_global, const StartSrc &src,
                                             float decay) {
    if (from_global)
        master_seed(tm_master + cx.lane_addr + 32 * cx.cq, src.state, src.delta, src.decay, src.j0, src.j1, src.st,
                    src.off + 32 * cx.cq);
    float ss = 0.f;
#pragma unroll
    for (int piece = 0; piece < 2; ++piece) {       // 16 columns at a time keeps the transient registers few
        uint32_t r[16];
        const uint32_t taddr = tm_master + cx.lane_addr + 32 * cx.cq + 16 * piece;
        TMEM_LD16(taddr, r);
        tmem_wait_ld();
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
            uint32_t pk[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float v0 = __uint_as_float(r[8 * ch + 2 * u]), v1 = __uint_as_float(r[8 * ch + 2 * u + 1]);
                if (SUMSQ) ss = fmaf(v0, v0, fmaf(v1, v1, ss));
                pk[u] = pack_bf16(v0, v1);
            }
            *reinterpret_cast<uint4 *>(cx.smem + OFF_H + tile_off(cx.c, 4 * cx.cq + 2 * piece + ch)) =
                make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * decay);
        TMEM_ST16(taddr, r);
    }
    tmem_wait_st();
    return ss;
}

// Copy this thread's part of a master from TMEM to global memory (final state of a sequence).
__device__ __forceinline__ void master_store(const Ctx &cx, uint32_t tm_master, float *grow) {
    uint32_t r[32];
    TMEM_LD32(tm_master + cx.lane_addr + 32 * cx.cq, r);
    tmem_wait_ld();
#pragma unroll
    for (int i = 0; i < 8; ++i)
        *reinterpret_cast<float4 *>(grow + 32 * cx.cq + 4 * i) =
            make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]), __uint_as_float(r[4 * i + 2]),
                        __uint_as_float(r[4 * i + 3]));
}

// Masked score epilogue: S (TMEM, fp32) -> P (packed bf16 pairs, written over the first 16 of this thread's own
// 32 score columns).  Keys j = 32 cq + i, token c = 32 q + l: blocks above the diagonal are zero, blocks below
// it need no mask.  The factor is the tile-wide constant pf, or per key (strongly decaying tiles, and the pass
// whose P multiplies the unweighted V).
enum { PF_CONST = 0, PF_TABLE = 1, PF_EXACT = 2 };   // tile-wide constant | 2^-G_j from the table | 2^(ac_c - G_j) per element
template <int MODE, bool DIAG>
__device__ __forceinline__ void p_block(const Ctx &cx, const GateScalars *gs, uint32_t taddr, float pf, float ac_c) {
    const uint64_t pf2 = f2_pack(pf, pf);
#pragma unroll
    for (int piece = 0; piece < 2; ++piece) {
        uint32_t r[16], pk[8];
        TMEM_LD16(taddr + 16 * piece, r);
        tmem_wait_ld();
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i0 = 16 * piece + 2 * u;
            uint64_t f2 = pf2;
            if (MODE == PF_TABLE) {
                const float2 z = *reinterpret_cast<const float2 *>(&gs->iz[32 * cx.cq + i0]);
                f2 = f2_pack(z.x, z.y);
            } else if (MODE == PF_EXACT) {
                f2 = f2_pack(ex2_fast(fminf(ac_c - cx.sc->G2cur[32 * cx.cq + i0], 126.f)),
                             ex2_fast(fminf(ac_c - cx.sc->G2cur[32 * cx.cq + i0 + 1], 126.f)));
            }
            float p0, p1;
            f2_unpack(f2_mul(f2_pack(__uint_as_float(r[2 * u]), __uint_as_float(r[2 * u + 1])), f2), p0, p1);
            if (DIAG) {                     // keys i <= l are visible
                p0 = (i0 <= cx.l) ? p0 : 0.f;
                p1 = (i0 + 1 <= cx.l) ? p1 : 0.f;
            }
            pk[u] = pack_bf16(p0, p1);
        }
        TMEM_ST8(taddr + 8 * piece, pk);
    }
}
__device__ __forceinline__ void p_epilogue(const Ctx &cx, const GateScalars *gs, int mode, float pf, float ac_c) {
    const uint32_t taddr = cx.tmem + TM_S + cx.lane_addr + 32 * cx.cq;
    if (cx.cq > cx.q) {
        uint32_t z[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) z[i] = 0u;
        TMEM_ST8(taddr, z);
        TMEM_ST8(taddr + 8, z);
    } else if (cx.cq == cx.q) {
        if (mode == PF_CONST) p_block<PF_CONST, true>(cx, gs, taddr, pf, ac_c);
        else if (mode == PF_TABLE) p_block<PF_TABLE, true>(cx, gs, taddr, pf, ac_c);
        else p_block<PF_EXACT, true>(cx, gs, taddr, pf, ac_c);
    } else {
        if (mode == PF_CONST) p_block<PF_CONST, false>(cx, gs, taddr, pf, ac_c);
        else if (mode == PF_TABLE) p_block<PF_TABLE, false>(cx, gs, taddr, pf, ac_c);
        else p_block<PF_EXACT, false>(cx, gs, taddr, pf, ac_c);
    }
    tmem_wait_st();
}

// Scale the 128 rows of a bf16 operand tile in place by per-row factors (each thread takes four 16-byte groups).
__device__ __forceinline__ void scale_rows(unsigned char *tile, const float *factor, int tid) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int qi = tid + CT * i;               // 16-byte group index in the 32 KB tile
        const float f = factor[(qi & 1023) >> 3];  // row of this group
        uint4 v = *reinterpret_cast<const uint4 *>(tile + qi * 16);
        uint32_t *pv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
        for (int u = 0; u < 4; ++u) pv[u] = pack_bf16(bf16_lo(pv[u]) * f, bf16_hi(pv[u]) * f);
        *reinterpret_cast<uint4 *>(tile + qi * 16) = v;
    }
}

// Inclusive scan over the tile's 128 tokens (threads 0..127 = warps 0..3, one token each) of the affine maps
// s -> a s + b, composed in token order; returns the map's value at `seed`.  `slot` selects the carry row.
__device__ __forceinline__ float affine_scan(const Ctx &cx, float a, float b, float seed, int slot) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float pa = __shfl_up_sync(0xffffffffu, a, o), pb = __shfl_up_sync(0xffffffffu, b, o);
        if (cx.l >= o) {
            b = fmaf(a, pb, b);
            a *= pa;
        }
    }
    // carries of whole warps go through shared memory
    float *ca = cx.sc->carry[slot][0], *cb = cx.sc->carry[slot][1];
    if (cx.l == 31) {
        ca[cx.q] = a;
        cb[cx.q] = b;
    }
#ifdef GKA_TC_TIMING
    if (cx.tid == 0) TRACE(0, 25);
#endif
    asm volatile("bar.sync 2, 128;" ::: "memory");
#ifdef GKA_TC_TIMING
    if (cx.tid == 0) TRACE(0, 26);
#endif
    float s = seed;
    for (int w = 0; w < cx.q; ++w) s = fmaf(ca[w], s, cb[w]);
    return fmaf(a, s, b);
}

// What a phase needs to know about a tile; recomputed from the tile's first chunk index at the start of every
// phase instead of being carried in registers through the solve loop.
struct TileInfo {
    int seq, n, ntok, m_next, b, h;
    bool run_start, seq_end;
    size_t tok0;
    long long f;
    const float *seq_state;    // caller's initial state of the tile's sequence, or nullptr
    bool chained;              // the run starts inside a sequence: its start state comes through the summaries
};
__device__ __forceinline__ TileInfo tile_info(const FwdArgs &a, int item, long long f_lo, int n_mine, int m) {
    const WorkPlan &P = a.plan;
    TileInfo t;
    t.f = f_lo + m;
    const unsigned fu = (unsigned)t.f;         // the chunk list is shorter than 2^31 (checked on the host)
    t.seq = (int)P.divN.div(fu);
    t.n = (int)(fu - (unsigned)t.seq * (unsigned)P.N);
    const int b = (int)a.divH.div((unsigned)t.seq), h = t.seq - b * a.heads;
    t.b = b;
    t.h = h;
    const bool two = (t.n + 1 < P.N) && (m + 1 < n_mine);
    t.ntok = min(two ? 2 * kChunk : kChunk, a.T - t.n * kChunk);   // the last chunk of a sequence may be short
    t.m_next = m + (two ? 2 : 1);
    t.tok0 = ((size_t)b * a.T + (size_t)t.n * kChunk) * a.heads + h;
    t.run_start = (m == 0) || (t.n == 0);
    t.seq_end = (t.n + (two ? 2 : 1) == P.N);
    t.seq_state = a.state_in ? a.state_in + (size_t)t.seq * state_floats(D, D) : nullptr;
    t.chained = t.run_start && t.n != 0;
    return t;
}

// EXTRA: the instantiation that also serves write strengths, the alpha-connection and the solve-only result; the
// plain forward runs the other one, whose code those options do not touch.
template <bool EXTRA>
__global__ void __launch_bounds__(kThreadsTile, 1)
fwd_tile_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmO, FwdArgs a) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_bars[BAR_COUNT];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    unsigned char *smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    const int tid = threadIdx.x;

    if (tid == 0) {
        s_abort = 0;
#ifdef GKA_TC_TIMING
        s_ttrace_n[0] = s_ttrace_n[1] = 0;
#endif
        for (int i = 0; i < BAR_COUNT; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s_bars[i])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&s_tmem_base))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = s_tmem_base;
    const uint32_t bars = smem_u32(&s_bars[0]);
    TileScalars *sc = reinterpret_cast<TileScalars *>(smem + OFF_SC);
    if (tid == 0) *reinterpret_cast<volatile int *>(&sc->stop) = 0;
    __syncthreads();

    const WorkPlan &P = a.plan;
    const int item = blockIdx.x;
    const long long f_lo = P.lo(item), f_hi = P.lo(item + 1);
    const int n_mine = (int)(f_hi - f_lo);          // chunks of this block

    if (tid >= CT) {
        // ================================ MMA issuing thread ================================
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsIssuer));
        if ((tid >> 5) == (CT >> 5) && n_mine > 0) {
            // ---- helper warp: the gate scalars of every tile, one tile ahead of the compute warps (cumulative log2
            // decay by a scan over the tile's tokens, 32 at a time)
            const int lane = tid & 31;
            const float *const beta_h = EXTRA ? a.beta : nullptr;
            const float *const alpha_h = EXTRA ? a.alpha : nullptr;
            int t = 0;
            for (int m = 0; m < n_mine; ++t) {
                const TileInfo ti = tile_info(a, item, f_lo, n_mine, m);
                // the buffer was last read by tile t - 2: wait for the compute warps to start tile t - 1 (they arrive on
                // this barrier at the start of every tile that has a successor, and once more if they stop early)
                if (t >= 2) {
                    asm volatile("bar.sync 4, 544;" ::: "memory");
                    if (*reinterpret_cast<const volatile int *>(&sc->stop)) break;
                }
                GateScalars *g = &sc->g[t & 1];
                float run = 0.f;
#pragma unroll 1
                for (int grp = 0; grp < 4; ++grp) {
                    const int cc = 32 * grp + lane;
                    const bool in = cc < ti.ntok;       // tokens past the tile: no decay, unit lambda / strengths
                    const size_t idx = ti.tok0 + (size_t)cc * a.heads;
                    const float gv = in ? __ldg(a.gate + idx) : 1.f;
                    const float lamv = in ? __ldg(a.lam + idx) : 1.f;
                    const float bv = (beta_h && in) ? __ldg(beta_h + idx) : 1.f;
                    const float av = (alpha_h && in) ? __ldg(alpha_h + idx) : 1.f;
                    const float lgc = fmaxf(log2f(gv), -115.f);
                    float incl = lgc;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const float up = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= o) incl += up;
                    }
                    const float G2c = run + incl;
                    run += __shfl_sync(0xffffffffu, incl, 31);
                    const float mc = fmaxf(G2c, -60.f);
                    g->lg[cc] = lgc;
                    g->G2[cc] = G2c;
                    g->ac[cc] = G2c - mc;
                    g->zt[cc] = exp2f(mc);
                    g->iz[cc] = exp2f(-mc);
                    g->lam[cc] = lamv;
                    g->sb[cc] = sqrtf(fmaxf(bv, 0.f));
                    g->al[cc] = av;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bars + 8 * (BAR_G0 + (t & 1)));
                m = ti.m_next;
            }
        }
        if ((tid >> 5) == (CT >> 5) + 2 && n_mine > 0) {     // one warp takes the requests; its lane 0 issues
            const uint32_t base14 = (smem_u32(smem) >> 4) & 0x3FFF;
            for (;;) {
                asm volatile("bar.sync 3, 544;" ::: "memory");   // the compute threads' sync_post
                const int req = *reinterpret_cast<const volatile int *>(&sc->req_op);
                if ((req & 0xFF) == OP_EXIT) break;
                if ((tid & 31) == 0) {
                    TRACE_HEAVY(1, 32 + (req & 0xFF));
                    fence_after();
                    issuer_run(req, base14, tmem, bars);
                    TRACE_HEAVY(1, 48 + (req & 0xFF));
                }
                __syncwarp();
            }
        }
    } else {
        // ================================= compute threads =================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsCompute));
        Ctx cx;
        cx.tid = tid;
        cx.l = tid & 31;
        cx.q = (tid >> 5) & 3;
        cx.cq = tid >> 7;
        cx.c = 32 * cx.q + cx.l;
        cx.lane_addr = (uint32_t)(32 * cx.q) << 16;
        cx.smem = smem;
        cx.sc = sc;
        cx.bars = bars;
        cx.tmem = tmem;
        cx.abort_addr = smem_u32(&s_abort);
        const int c = cx.c, cq = cx.cq, l = cx.l;
        const uint32_t sbase = smem_u32(smem);
        const size_t st = state_floats(D, D);
        const bool adaptive = (a.flags & GKA_FLAG_ADAPTIVE_LAMBDA) != 0;
        const bool solve_only = EXTRA && a.solve_only != 0;   // the result is the solve itself: no V, no U, no output product
        const float *const beta_p = EXTRA ? a.beta : nullptr;
        const float *const alpha_p = EXTRA ? a.alpha : nullptr;
        const bool mix = alpha_p != nullptr && !solve_only;   // alpha-connection: the read uses alpha x + (1 - alpha) q
        uint32_t ph_a = 0, ph_b = 0;
        // first item of the chain of summaries behind this block's start state: the one whose range holds the
        // start of the sequence (its last run begins there, whatever sequence the item itself started in)
        int chain_j0 = item;
        if (n_mine > 0 && P.cut_in(item)) {
            const long long seq_start = (f_lo / P.N) * P.N;
            chain_j0 = item - 1;
            while (P.lo(chain_j0) > seq_start) --chain_j0;
        }

        // K (or V) tile of flat chunk f: 128 rows starting at the chunk's first token; rows past the tile's
        // tokens belong to later tokens (or are zero-filled past the end of the sequence) and are never used
        auto issue_tma = [&](const CUtensorMap *map, long long f, uint32_t dst, int bar_idx) {
            const unsigned fu = (unsigned)f;
            const int seq = (int)P.divN.div(fu), n = (int)(fu - (unsigned)seq * (unsigned)P.N);
            const int b = (int)a.divH.div((unsigned)seq), h = seq - b * a.heads;
            const int y = n * kChunk;
            const uint32_t bar = bars + 8 * bar_idx;
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(32768u) : "memory");
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int x = h * D + 64 * hf;
                asm volatile(
                    "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::
                        "r"(sbase + dst + 16384 * hf), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(b), "r"(bar)
                    : "memory");
            }
        };

        if (tid == 0 && n_mine > 0) issue_tma(&tmK, f_lo, OFF_K0, BAR_K0);
        // launched as a programmatic dependent of the summary kernel: everything above overlapped its tail; the
        // summaries are read by these threads only (no effect when there is no such dependency)
        asm volatile("griddepcontrol.wait;" ::: "memory");

        int tile = 0;
        bool stopped_early = false;
        for (int m = 0; m < n_mine; ++tile) {       // m: index of the tile's first chunk inside the block's range
            const int stage = tile & 1;
            const uint32_t off_k = stage ? OFF_K1 : OFF_K0;
            bool valid, clamped;
            float pf;

            // ======================= phase 1: operands, state pass, Frobenius norms =======================
            {
                const TileInfo ti = tile_info(a, item, f_lo, n_mine, m);
                const int ntok = ti.ntok;
                valid = c < ntok;
                // the previous tile is finished: the q / V buffer and the other K stage are free (issued by a thread
                // that has no part in the gate scan below, which every warp waits for)
                if (tid == NT) {
                    issue_tma(&tmQ, ti.f, OFF_V, BAR_V);
                    if (ti.m_next < n_mine)
                        issue_tma(&tmK, f_lo + ti.m_next, stage ? OFF_K0 : OFF_K1, stage ? BAR_K0 : BAR_K1);
                }
                // ---- the tile's gate scalars were prepared by the helper warp during the previous tile
                GateScalars *const gs = &sc->g[stage];
                if (tile >= 1 && ti.m_next < n_mine) asm volatile("bar.arrive 4, 544;" ::: "memory");   // the other buffer is free
                wait_bar(cx, stage ? BAR_G1 : BAR_G0, (uint32_t)((tile >> 1) & 1));
                if (tid < NT) sc->G2cur[c] = gs->G2[c];      // published by the barriers below, long before the solve loop
                TSTAMP(23);
                // ---- K tile has landed (it was fetched during the previous tile): Gram matrix under the set-up
                wait_bar(cx, stage ? BAR_K1 : BAR_K0, (uint32_t)((tile >> 1) & 1));
                if (beta_p) {      // beta k k^T is the plain write of sqrt(beta) k: rescale the key rows in place
                    cta_sync();
                    scale_rows(smem + off_k, gs->sb, tid);
                    fence_async_smem();
                }
                const float Glast = gs->G2[ntok - 1];
                clamped = Glast < -60.f;                      // the tile decays below 2^-60: per-element factors
                pf = exp2f(-fmaxf(Glast, -60.f));             // Gamma[c][j] / zt_c = pf * w_j otherwise
                const float decay = exp2f(Glast);             // zeta of the whole tile

                // ---- w o K (same swizzled positions as K), rows past the tile weigh nothing
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int qi = tid + CT * i;               // 16-byte group index in the 32 KB tile
                    const int j = (qi & 1023) >> 3;            // key row of this group
                    uint4 v = *reinterpret_cast<const uint4 *>(smem + off_k + qi * 16);
                    const float wj = (j < ntok) ? exp2f(Glast - gs->G2[j]) : 0.f;
                    uint32_t *pv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
                    for (int u = 0; u < 4; ++u) pv[u] = pack_bf16(bf16_lo(pv[u]) * wj, bf16_hi(pv[u]) * wj);
                    *reinterpret_cast<uint4 *>(smem + OFF_KW + qi * 16) = v;
                }
                TSTAMP(2);
                // the Gram matrix runs under the state pass (the weighting above would fight it for shared memory)
                sync_post(cx, OP_GRAM | (stage ? OPF_STAGE : 0));
                TSTAMP(0);

                // ---- H master, one pass: ||H_0||^2, bf16 copy, scale by the tile's decay
                {
                    const StartSrc src = {(ti.chained && a.start_from_scan) ? a.ws.start + (size_t)item * st : ti.seq_state,
                                          a.ws.delta, a.ws.decay, (ti.chained && !a.start_from_scan) ? chain_j0 : 0,
                                          (ti.chained && !a.start_from_scan) ? item : 0, st, (size_t)c * D};
                    float hs = master_pass<true>(cx, tmem + TM_H, ti.run_start, src, decay);
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) hs += __shfl_xor_sync(0xffffffffu, hs, o);
                    if (l == 0) sc->red[tid >> 5] = hs;
                }
                fence_async_smem();
                fence_before();
                sync_post(cx, OP_FROB | (stage ? OPF_STAGE : 0));
                TSTAMP(3);
                wait_bar(cx, BAR_A, ph_a);
                ph_a ^= 1u;
                fence_after();
                TSTAMP(4);

                // ---- chunk-wise Frobenius norms: per key, k_j^T H_0 k_j and the decayed squared Gram entries of
                // the earlier keys.  Thread = (key j = c, 32 columns).
                {
                    float kh = 0.f, gsum = 0.f;
#pragma unroll
                    for (int piece = 0; piece < 2; ++piece) {
                        uint32_t r[16];
                        TMEM_LD16(tmem + TM_Y + cx.lane_addr + 32 * cq + 16 * piece, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int ch = 0; ch < 2; ++ch) {
                            const uint4 kv =
                                *reinterpret_cast<const uint4 *>(smem + off_k + tile_off(c, 4 * cq + 2 * piece + ch));
                            const uint32_t *pk = reinterpret_cast<const uint32_t *>(&kv);
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                kh = fmaf(__uint_as_float(r[8 * ch + 2 * u]), bf16_lo(pk[u]), kh);
                                kh = fmaf(__uint_as_float(r[8 * ch + 2 * u + 1]), bf16_hi(pk[u]), kh);
                            }
                        }
                    }
                    if (cq <= cx.q) {
                        const float G2j = gs->G2[c];
                        const int lim = (cq == cx.q) ? l : 32;   // keys i < lim come earlier, i == lim is the key itself
                        float gd = 0.f;                          // the key's own squared norm
                        uint64_t acc2 = 0ull;
#pragma unroll
                        for (int piece = 0; piece < 2; ++piece) {
                            uint32_t r[16];
                            TMEM_LD16(tmem + TM_S + cx.lane_addr + 32 * cq + 16 * piece, r);
                            tmem_wait_ld();
                            if (!clamped) {         // sum_i g_i^2 2^-G_i over the earlier keys, times 2 2^G_j afterwards
#pragma unroll
                                for (int u = 0; u < 8; ++u) {
                                    const int ii = 16 * piece + 2 * u;
                                    const float g0 = __uint_as_float(r[2 * u]), g1 = __uint_as_float(r[2 * u + 1]);
                                    if (ii == lim) gd = g0 * g0;
                                    if (ii + 1 == lim) gd = g1 * g1;
                                    const uint64_t gg = f2_pack(ii < lim ? g0 : 0.f, ii + 1 < lim ? g1 : 0.f);
                                    const float2 z = *reinterpret_cast<const float2 *>(&gs->iz[32 * cq + ii]);
                                    acc2 = f2_fma(f2_mul(gg, gg), f2_pack(z.x, z.y), acc2);
                                }
                            } else {
#pragma unroll
                                for (int i = 0; i < 16; ++i) {
                                    const int ii = 16 * piece + i;
                                    const float g = __uint_as_float(r[i]);
                                    const float g2 = g * g;
                                    if (ii < lim) gsum = fmaf(2.f * ex2_fast(G2j - gs->G2[32 * cq + ii]), g2, gsum);
                                    else if (ii == lim) gd = g2;
                                }
                            }
                        }
                        float a0, a1;
                        f2_unpack(acc2, a0, a1);
                        gsum = fmaf(2.f * ex2_fast(G2j), a0 + a1, gsum) + gd;
                    }
                    sc->part[0][cq][c] = kh;
                    sc->part[1][cq][c] = gsum;
                }
                fence_before();
                cta_sync();
                // the H master is final for this tile
                if (ti.seq_end && a.state_out)
                    master_store(cx, tmem + TM_H, a.state_out + (size_t)ti.seq * st + (size_t)c * D);
                TSTAMP(5);

                // ---- f_c by an affine scan (s_c = gamma_c^2 s_{c-1} + d_c, s_{-1} = ||H_0||^2), Chebyshev set-up
                if (tid < NT) {
                    float hh = 0.f;
#pragma unroll
                    for (int i = 0; i < 16; ++i) hh += sc->red[i];
                    const float kh = (sc->part[0][0][c] + sc->part[0][1][c]) + (sc->part[0][2][c] + sc->part[0][3][c]);
                    const float gsum = (sc->part[1][0][c] + sc->part[1][1][c]) + (sc->part[1][2][c] + sc->part[1][3][c]);
                    const float dc = fmaf(2.f * exp2f(gs->G2[c]), kh, gsum);
                    const float s = affine_scan(cx, exp2f(2.f * gs->lg[c]), dc, hh, 1);
                    const float fc = sqrtf(fmaxf(s, 0.f));
                    float lamc = gs->lam[c];
                    if (adaptive) lamc *= fc;
                    const float Lpm = fc + 2.f * lamc;
                    const float rho = fc / Lpm;
                    sc->lam[c] = lamc;
                    sc->rho2[c] = rho * rho;
                    sc->s0[c] = 2.f / Lpm;
                    if (a.fro_out && valid) a.fro_out[ti.tok0 + (size_t)c * a.heads] = fc;
                }
                wait_bar(cx, BAR_V, solve_only ? (uint32_t)(tile & 1) : 0u);   // q tile has landed (V shares the barrier)
                // the previous tile's output stores have read the X' buffer, which x_0 is about to overwrite
                if (tid == 32) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                cta_sync();                    // the set-up values are published
            }

            // ======================= phase 2: Algorithm 1 on the whole tile =======================
            {
                // per-token scalars (this thread's token), x_0 = 2 q / (L + mu)
                const float s0 = sc->s0[c], rho2 = sc->rho2[c], lamc = sc->lam[c], ztc = sc->g[stage].zt[c], acc_c = sc->g[stage].ac[c];
                const unsigned char *qrow = smem + OFF_V;      // q tile: this thread reads row c, its 4 groups of 8 channels
                uint64_t x2[16];   // the iterate (fp32 pairs), scaled by zt_c (the recurrence is linear), as the operand needs it
                uint64_t xp2[16];  // the previous iterate
                {
                    const float x0s = valid ? s0 * ztc : 0.f;  // tokens past the tile stay zero
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        const uint4 qv = *reinterpret_cast<const uint4 *>(qrow + tile_off(c, 4 * cq + ch));
                        const uint32_t *qq = reinterpret_cast<const uint32_t *>(&qv);
                        uint32_t pk[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const float xa = x0s * bf16_lo(qq[u]), xb = x0s * bf16_hi(qq[u]);
                            x2[4 * ch + u] = f2_pack(xa, xb);
                            xp2[4 * ch + u] = 0ull;              // x_{-1} = 0 (Algorithm 1)
                            pk[u] = pack_bf16(xa, xb);
                        }
                        *reinterpret_cast<uint4 *>(smem + OFF_X + tile_off(c, 4 * cq + ch)) =
                            make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
                const int rq = (stage ? OPF_STAGE : 0) | (clamped ? OPF_PLAIN_K : 0);
                fence_async_smem();
                fence_before();
                // after the last update: scores for the output (posted later when the iterate is still to be mixed with q)
                const int op_last = (solve_only || mix) ? OP_NONE : OP_ITER1_LAST;
                sync_post(cx, (a.n_iter == 0 ? op_last : OP_ITER1) | rq);
                TSTAMP(6);

                float omega = 2.f;
                for (int it = 0; it < a.n_iter; ++it) {
                    // weight schedule and this token's coefficients, while the scores are computed
                    omega = 4.f / (4.f - rho2 * omega);
                    const float sigma = s0 * omega, beta = omega - 1.f;
                    const float cfx = valid ? sigma * ztc : 0.f, cfz = sigma * lamc;
                    const float cfa = 1.f + beta - cfz;     // x_{i+1} = cfa x_i - beta x_{i-1} + cfx (q - H_c x_i)
                    const uint64_t cfx2 = f2_pack(cfx, cfx), cfa2 = f2_pack(cfa, cfa), nbeta2 = f2_pack(-beta, -beta);
                    wait_bar(cx, BAR_A, ph_a);
                    ph_a ^= 1u;
                    fence_after();
                    TSTAMP(7);
                    p_epilogue(cx, nullptr, clamped ? PF_EXACT : PF_CONST, pf, acc_c);
                    fence_before();
                    sync_post(cx, OP_ITER2 | rq);
                    TSTAMP(8);

                    wait_bar(cx, BAR_B, ph_b);
                    ph_b ^= 1u;
                    fence_after();
                    TSTAMP(9);
                    // x_{i+1} = cfa x_i - beta x_{i-1} + cfx (q - H_c x_i) overwrites x_{i-1}; the arrays are swapped after
                    auto x_epilogue = [&](uint64_t(&cur)[16], uint64_t(&prv)[16]) {
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch) {    // 8 channels at a time keeps the transient registers few
                            uint32_t r[8];
                            TMEM_LD8(tmem + TM_Y + cx.lane_addr + 32 * cq + 8 * ch, r);
                            const uint4 qv = *reinterpret_cast<const uint4 *>(qrow + tile_off(c, 4 * cq + ch));
                            const uint32_t *qq = reinterpret_cast<const uint32_t *>(&qv);
                            tmem_wait_ld();
                            uint32_t pk[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                const int i = 4 * ch + u;
                                const uint64_t t2 = f2_sub(f2_pack(bf16_lo(qq[u]), bf16_hi(qq[u])),
                                                           f2_pack(__uint_as_float(r[2 * u]), __uint_as_float(r[2 * u + 1])));
                                prv[i] = f2_fma(cfx2, t2, f2_fma(cfa2, cur[i], f2_mul(nbeta2, prv[i])));
                                float xa, xb;
                                f2_unpack(prv[i], xa, xb);
                                pk[u] = pack_bf16(xa, xb);
                            }
                            *reinterpret_cast<uint4 *>(smem + OFF_X + tile_off(c, 4 * cq + ch)) =
                                make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        }
                    };
                    x_epilogue(x2, xp2);
#pragma unroll
                    for (int i = 0; i < 16; ++i) {      // the new iterate becomes x2 again
                        const uint64_t tmp = x2[i];
                        x2[i] = xp2[i];
                        xp2[i] = tmp;
                    }
                    fence_async_smem();
                    fence_before();
                    sync_post(cx, (it + 1 == a.n_iter ? op_last : OP_ITER1) | rq);
                    TSTAMP(10);
                }
                if (solve_only) {
                    // the solve is the result: x_c = x'_c / zt_c as bf16 into the X' buffer (no product reads it any
                    // more), stored by TMA after the tile's last barrier
                    const float inv = sc->g[tile & 1].iz[c];
                    auto stage_x = [&](const uint64_t(&x)[16]) {
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch) {
                            uint32_t pk[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                float xa, xb;
                                f2_unpack(x[4 * ch + u], xa, xb);
                                pk[u] = pack_bf16(xa * inv, xb * inv);
                            }
                            *reinterpret_cast<uint4 *>(smem + OFF_X + tile_off(c, 4 * cq + ch)) =
                                make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        }
                    };
                    stage_x(x2);
                    fence_async_smem();
                }
                if (mix) {
                    // alpha-connection (Section 4.4): X' <- zt (alpha x + (1 - alpha) q) = alpha x' + (1 - alpha) zt q
                    const float alc = sc->g[tile & 1].al[c];
                    auto mix_x = [&](const uint64_t(&x)[16]) {
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch) {
                            const uint4 qv = *reinterpret_cast<const uint4 *>(qrow + tile_off(c, 4 * cq + ch));
                            const uint32_t *qq = reinterpret_cast<const uint32_t *>(&qv);
                            uint32_t pk[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                float xa, xb;
                                f2_unpack(x[4 * ch + u], xa, xb);
                                const float qa = valid ? ztc * bf16_lo(qq[u]) : 0.f, qb = valid ? ztc * bf16_hi(qq[u]) : 0.f;
                                pk[u] = pack_bf16(fmaf(alc, xa - qa, qa), fmaf(alc, xb - qb, qb));
                            }
                            *reinterpret_cast<uint4 *>(smem + OFF_X + tile_off(c, 4 * cq + ch)) =
                                make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        }
                    };
                    mix_x(x2);
                    fence_async_smem();
                    fence_before();
                    sync_post(cx, OP_ITER1_LAST | rq);
                }
            }

            // ======================= phase 3: last score pass, output, U advance =======================
            TSTAMP(17);
            {
                int mm = m;
                asm volatile("" : "+r"(mm));                   // recompute the tile's description
                const TileInfo ti = tile_info(a, item, f_lo, n_mine, mm);
                const GateScalars *const gs = &sc->g[tile & 1];
                if (!solve_only) {
                    // q is no longer needed: its buffer takes the V tile
                    if (tid == 0) issue_tma(&tmV, ti.f, OFF_V, BAR_V);
                    // while the scores of the final iterate are computed: U master pass (bf16 copy into the H buffer, which
                    // no pending product reads; scale by the tile's decay)
                    const StartSrc src = {(ti.chained && a.start_from_scan) ? a.ws.start + (size_t)item * st : ti.seq_state,
                                          a.ws.delta, a.ws.decay, (ti.chained && !a.start_from_scan) ? chain_j0 : 0,
                                          (ti.chained && !a.start_from_scan) ? item : 0, st, (size_t)D * D + (size_t)c * D};
                    master_pass<false>(cx, tmem + TM_U, ti.run_start, src, exp2f(gs->G2[ti.ntok - 1]));
                    fence_async_smem();
                    fence_before();
                    sync_post(cx, OP_OUT_U0);
                    wait_bar(cx, BAR_A, ph_a);
                    ph_a ^= 1u;
                    fence_after();
                    TSTAMP(15);
                    p_epilogue(cx, gs, clamped ? PF_EXACT : PF_TABLE, pf, gs->ac[c]);   // this P multiplies the unweighted V
                    fence_before();
                    TSTAMP(16);
                    // O = X' U_0^T + P V (the H buffer holds U_0 since the last score pass), U advance
                    wait_bar(cx, BAR_V, 1u);                       // V tile has landed
                    if (beta_p) {  // beta v k^T with sqrt(beta) k already in place: the value rows take the other sqrt(beta)
                        scale_rows(smem + OFF_V, gs->sb, tid);
                        fence_async_smem();
                    }
                    sync_post(cx, OP_OUT | (stage ? OPF_STAGE : 0));
                    TSTAMP(11);
                    wait_bar(cx, BAR_A, ph_a);
                    ph_a ^= 1u;
                    fence_after();
                    TSTAMP(12);
                    // O as bf16 into the X' buffer (no product reads it any more), stored by TMA after the tile's last barrier
#pragma unroll
                    for (int piece = 0; piece < 2; ++piece) {
                        uint32_t r[16];
                        TMEM_LD16(tmem + TM_Y + cx.lane_addr + 32 * cq + 16 * piece, r);
                        tmem_wait_ld();
                        uint32_t pk[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u)
                            pk[u] = pack_bf16(__uint_as_float(r[2 * u]), __uint_as_float(r[2 * u + 1]));
                        *reinterpret_cast<uint4 *>(smem + OFF_X + tile_off(c, 4 * cq + 2 * piece)) =
                            make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        *reinterpret_cast<uint4 *>(smem + OFF_X + tile_off(c, 4 * cq + 2 * piece + 1)) =
                            make_uint4(pk[4], pk[5], pk[6], pk[7]);
                    }
                    fence_async_smem();
                    TSTAMP(13);
                    wait_bar(cx, BAR_B, ph_b);     // U advance done: every tensor-core read of this tile's buffers is done
                    ph_b ^= 1u;
                    fence_after();
                    if (ti.seq_end && a.state_out)
                        master_store(cx, tmem + TM_U, a.state_out + (size_t)ti.seq * st + (size_t)D * D + (size_t)c * D);
                }
                fence_before();
                if (tid == 0) sc->stop = aborted(cx) ? 1 : 0;
                cta_sync();
                TSTAMP(14);
                if (tid == 32) {              // one box of 64 tokens x 64 channels per chunk and channel half
                    const int b = ti.b, h = ti.h;
                    for (int hh = 0; hh < (ti.ntok + kChunk - 1) / kChunk; ++hh)     // rows past the sequence are clipped
                        for (int hf = 0; hf < 2; ++hf)
                            asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];" ::
                                             "l"(reinterpret_cast<uint64_t>(&tmO)), "r"(h * D + 64 * hf),
                                         "r"((ti.n + hh) * kChunk), "r"(b), "r"(sbase + OFF_X + 16384 * hf + 8192 * hh)
                                         : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
                if (sc->stop) {               // the same decision in every thread
                    stopped_early = true;
                    break;
                }
                m = ti.m_next;
            }
        }
        if (stopped_early) asm volatile("bar.arrive 4, 544;" ::: "memory");   // releases the helper warp, which then sees the stop flag
        if (n_mine > 0) sync_post(cx, OP_EXIT);
        if (tid == 32) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // output stores are complete
    }

#ifdef GKA_TC_TIMING
    __syncthreads();
    if (blockIdx.x == 0 && tid < 2) g_ttrace_n[tid] = s_ttrace_n[tid];
#endif
    fence_before();
    __syncthreads();
    if (tid == 0 && s_abort != 0 && a.device_status) atomicExch(a.device_status, (int)GKA_ERR_TIMEOUT);
    if (tid < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
}

}  // namespace

cudaError_t launch_fwd_tile(const FwdArgs &a, cudaStream_t stream) {
    alignas(64) CUtensorMap tmK, tmV, tmQ, tmO;     // the output is stored chunk by chunk: boxes of 64 rows
    const int cols = a.heads * D;
    if (!make_tile_map(&tmK, a.k, a.B, a.T, cols, NT) || !make_tile_map(&tmV, a.v, a.B, a.T, cols, NT) ||
        !make_tile_map(&tmQ, a.q, a.B, a.T, cols, NT) || !make_tile_map(&tmO, a.out, a.B, a.T, cols, kChunk))
        return cudaErrorInvalidValue;
    const bool extra = a.beta != nullptr || a.alpha != nullptr || a.solve_only != 0;
    auto kernel = extra ? fwd_tile_kernel<true> : fwd_tile_kernel<false>;
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TILE_SMEM);
    if (err != cudaSuccess) return err;
    if (a.ev_start) cudaEventRecord(a.ev_start, stream);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)a.plan.G);
    cfg.blockDim = dim3(kThreadsTile);
    cfg.dynamicSmemBytes = TILE_SMEM;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.after_summary ? 1 : 0;
    err = cudaLaunchKernelEx(&cfg, kernel, tmK, tmV, tmQ, tmO, a);
    if (err != cudaSuccess) return err;
    if (a.ev_stop) cudaEventRecord(a.ev_stop, stream);
    return cudaGetLastError();
}

#ifdef GKA_TC_TIMING
extern "C" int gka_debug_tile_trace(long long *out /* 2 x 8192 */, int *counts /* 2 */) {
    if (cudaMemcpyFromSymbol(out, g_ttrace, sizeof(long long) * 2 * 8192) != cudaSuccess) return 1;
    if (cudaMemcpyFromSymbol(counts, g_ttrace_n, sizeof(int) * 2) != cudaSuccess) return 1;
    return 0;
}
#endif

}  // namespace gka
