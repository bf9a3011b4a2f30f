// tcgen05 / TMEM solve kernel of the chunk-wise GKA forward (bf16 operands, fp32 accumulation) for sm_100a.
//
// Input: for every tile of 128 consecutive tokens of a sequence, the bf16 copies of the tile-initial states
// H_0, U_0 and ||H_0||_F^2 (written by the state kernel, gka_tc_state.cu).  Tiles are independent problems.  One
// persistent thread block per SM keeps two tiles ("slots") in flight and runs them in opposite phases: while the
// tensor pipe works on the products of one slot, the CUDA cores run the fp32 update of the other.  A tile puts one
// token on each TMEM lane; every product of the chunk-wise form (Section 4.2.1; Algorithm 1 on the whole tile) is
// an M = 128 tile.
//
// Algorithm 1 in residual form.  With d_i = x_i - x_{i-1} (x_{-1} = 0, d_0 = x_0 = 2 q / (L + mu)) the update
// x_{i+1} = x_i + (omega_{i+1} - 1) d_i + (2 omega_{i+1} / (L + mu)) (q - A x_i) reads
//     r_i = r_{i-1} - A d_i  (r_{-1} = q),     d_{i+1} = beta d_i + sigma r_i,     x_{i+1} = x_i + d_{i+1},
// the same iterates in exact arithmetic.  The matrix is applied to the increment d_i, so the bf16 rounding of the
// tensor-core operand is relative to the (shrinking) increment and the iterate itself stays in fp32; the value
// added to x is the rounded operand, which keeps x and the residual consistent.  Per token c of the tile
//     A d = zeta_c H_0 d + sum_{j<=c} Gamma[c][j] k_j (k_j . d) + lambda_c d,     Gamma[c][j] = 2^(G_c - G_j),
// G the cumulative log2 gate in the tile.  The operand is E = -zt_c d_c in bf16 (zt_c = max(zeta_c, 2^-60)), the
// keys are staged as Khat_j = sqrt(beta_j) 2^(-G_j / 2) k_j, and the accumulator R starts as q:
//     S = E Khat^T,   P = S masked to j <= c (packed bf16, written over S in TMEM),   R += E H_0^T + P Khat
// leaves R = q - (A - lambda) x_i with no factor anywhere in the masked-score epilogue; the lambda term uses the
// fp32 iterate.  Tiles whose decay falls below 2^-60 keep unscaled keys and per-element factors instead.
// The read o_c = zeta_c U_0 x_c + sum_{j<=c} Gamma[c][j] v_j (k_j . x_c) uses the final iterate split into two
// bf16 terms (x is dominated by directions that U barely reads; a single bf16 rounding of x would swamp the rest).
// Chunk-wise Frobenius norms of Section 4.2.1 come from Khat H_0, the Gram matrix Khat Khat^T and an affine scan.
//
// On-chip layout.  Tensor memory (512 columns): one score tile S shared by the two slots (only one slot at a time
// is between its score product and the product that consumes the masked scores: the issuing thread hands S from
// slot to slot, which is also what keeps the slots in opposite phases), and per slot the fp32 accumulator R (128
// columns) and the operand E as packed bf16 (64 columns).  E and P feed the products from tensor memory, so a
// product reads only its B operand (keys, H_0, U_0, values) from shared memory and leaves half of the shared-memory
// bandwidth to everything else.  Shared memory per slot: keys, H_0 (later U_0), q (later V, then the result).
//
// Warp roles: 4 compute warps per slot, a thread owns one token (one TMEM lane) and all 128 channels of its
// iterate in registers; 4 score warps (one per TMEM lane quadrant) run the masked-score epilogue of both slots; one
// warp prepares the gate scalars one tile ahead; one thread per slot issues that slot's TMA stores and the loads that
// follow them; one thread issues every tcgen05.mma for both slots.  Requests to the issuing thread are counters in
// shared memory (one count per warp), completion comes back through tcgen05.commit mbarriers.  What bounds the
// iterations is the turn of a slot on the score tile (score product, epilogue, second product); stores to tensor
// memory (about 40 bytes per cycle per SM) are the scarce resource of the epilogues.
//
// Head dimension 64 arrives zero-extended to 128 channels (the upper TMA box reads zeros).  The kernel instantiated
// with HALF leaves out what the zero channels would contribute: contractions over the channels take four k-steps
// instead of eight, and the passes of the compute warps over the channels stop at channel 64.  Its turns on the score
// tile are shorter, so the masked-score epilogue weighs more: there the slot's compute warps, idle during the turn,
// convert the upper key blocks of their tokens and the score warps the lower ones.
#include <cuda.h>

#include "gka_common.cuh"
#include "gka_tc_mma.cuh"

namespace gka {
namespace {

using namespace tcu;

constexpr int NT = kTile;                  // tokens per tile: one per TMEM lane
constexpr int kSlots = 2;
constexpr int ST = 128;                    // compute threads per slot
constexpr int CT = kSlots * ST;            // compute threads
// Warpgroups: 0 = helpers (gate scalars, TMA: one warp per slot, MMA issue), 1 = score warps (the masked-score
// epilogue of both slots, one warp per TMEM lane quadrant), 2 and 3 = the compute warps of slot 0 and slot 1.
constexpr int kThreadsSolve = 256 + CT;
constexpr int kRegsLaunch = 128, kRegsCompute = 200, kRegsScore = 64, kRegsHelper = 48;   // register split after setmaxnreg
static_assert(kThreadsSolve * kRegsLaunch <= 65536, "launch registers");
static_assert(CT * kRegsCompute + 128 * kRegsScore + 128 * kRegsHelper <= kThreadsSolve * kRegsLaunch, "register split exceeds the launch allocation");

// ---- shared memory map (bytes; operand buffers 1024-byte aligned): three operand tiles per slot, then the scalars
constexpr uint32_t BUF_A = 0;                  // keys (Khat)
constexpr uint32_t BUF_B = kTileBytes;         // bf16 H_0, later U_0
constexpr uint32_t BUF_C = 2 * kTileBytes;     // q, later V, then the result tile
constexpr uint32_t SLOT_BYTES = 3 * kTileBytes;
constexpr uint32_t OFF_SC = kSlots * SLOT_BYTES;

struct GateScalars {       // per token of a tile, from the gates and the other per-token inputs alone
    float lg[NT];          // log2 gamma_c
    float G2[NT];          // cumulative log2 gate
    float ac[NT];          // G2_c - max(G2_c, -60): exponent correction of clamped tokens
    float zt[NT];          // clamped zeta_c
    float iz[NT];          // 1 / zt_c
    float lam[NT];         // lambda_c as given
    float al[NT];          // alpha_c (alpha-connection)
    float ks[NT];          // row factor of the staged keys: sqrt(beta_j) 2^(-G_j / 2), or sqrt(beta_j) alone when the tile decays below 2^-60
};
struct SlotScalars {
    GateScalars g[2];
    float carry[2][4];     // per-warp totals (a, b) of the affine scan
    int exact[2];          // the tile of gate buffer 0 / 1 decays below 2^-60 (per-element factors in the score epilogue)
};
constexpr uint32_t SC_BYTES = (sizeof(SlotScalars) + 127) / 128 * 128;
constexpr uint32_t SOLVE_SMEM = OFF_SC + kSlots * SC_BYTES + 1024;   // + slack for the 1024-byte alignment of the base
static_assert(SOLVE_SMEM + 2048 <= 232448, "shared memory budget");

// ---- TMEM columns: shared score accumulator S (P overwrites it in place); per slot the residual / output
// accumulator R and the bf16 operand E
constexpr uint32_t TM_S = 0;
__host__ __device__ constexpr uint32_t tm_r_of(int s) { return 128u + 128u * (uint32_t)s; }
__host__ __device__ constexpr uint32_t tm_e_of(int s) { return 384u + 64u * (uint32_t)s; }

enum {                 // per slot
    B_LD_K = 0,        // K tile has landed (TMA)
    B_LD_H,            // H_0 tile
    B_LD_Q,            // q tile
    B_LD_U,            // U_0 tile
    B_LD_V,            // V tile
    B_RDY_ST,          // compute warps -> TMA thread: the result tile is staged
    B_QF,              // compute warps -> TMA thread: q has been read, V may take its buffer
    B_MMA_S,           // tcgen05.commit: the Frobenius batch (Gram matrix, K H_0) is complete
    B_MMA_R,           // tcgen05.commit: accumulator-side batch complete
    B_GS0, B_GS1,      // gate scalars of buffer 0 / 1 are ready
    B_GF0, B_GF1,      // compute warps -> gate helper: buffer 0 / 1 is free
    B_PER_SLOT
};
constexpr int B_DRAIN = kSlots * B_PER_SLOT;   // every product is complete (before the tensor memory is given back)
constexpr int B_SC = B_DRAIN + 1;              // tcgen05.commit: a score product of either slot is complete (-> score warps)
constexpr int B_COUNT = B_SC + 1;

// Requests a slot makes to the issuing thread: every warp of the slot adds one to the slot's request counter in
// shared memory (a poll of both counters is one 40-cycle load, where a test of an mbarrier phase takes 100 cycles);
// request n of a slot is ready when its counter has reached 4 (n + 1).  In this order per tile:
// FROB, then n_iter times (ITER1, ITER2), then (unless the solve itself is the result) OUT_S, OUT_O
enum { OP_FROB = 0, OP_ITER1, OP_ITER2, OP_OUT_S, OP_OUT_O };

__device__ __forceinline__ bool aborted(uint32_t abort_addr) {
    int v;
    asm volatile("ld.volatile.shared.b32 %0, [%1];" : "=r"(v) : "r"(abort_addr) : "memory");
    return v != 0;
}
__device__ __forceinline__ void set_abort(uint32_t abort_addr) {
    asm volatile("st.volatile.shared.b32 [%0], %1;" ::"r"(abort_addr), "r"(1) : "memory");
}
// Bounded wait (about a second; the wait suspends in hardware between polls); once any wait of the block has given up
// every later wait returns at once, so the block runs to its end without further delays and reports
// GKA_ERR_TIMEOUT.  One compact loop in a single asm block: the wait is inlined at some thirty places.
__device__ __forceinline__ void wait_bar(uint32_t bar, uint32_t parity, uint32_t abort_addr) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .u32 n, ab;\n\t"
        "mov.u32 n, 0;\n\t"
        "ld.volatile.shared.b32 ab, [%4];\n\t"
        "setp.ne.u32 p, ab, 0;\n\t"
        "@p bra WAIT_DONE;\n"
        "WAIT_LOOP:\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "@p bra WAIT_DONE;\n\t"
        "add.u32 n, n, 1;\n\t"
        "setp.lt.u32 q, n, 200000;\n\t"
        "@q bra WAIT_LOOP;\n"
        "WAIT_DONE:\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(5000u), "r"(abort_addr)
        : "memory");
    if (!ok) set_abort(abort_addr);
}
// one count per warp on a shared-memory counter, after every lane's writes and fences (release)
__device__ __forceinline__ void warp_post(uint32_t addr, int lane) {
    __syncwarp();
    if (lane == 0) asm volatile("red.release.cta.shared::cta.add.u32 [%0], 1;" ::"r"(addr) : "memory");
}
// one arrival per warp, after every lane's writes and fences
__device__ __forceinline__ void warp_arrive(uint32_t bar, int lane) {
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
}

struct TileInfo {
    int seq, n, b, h, ntok;
    size_t tok0;
};
__device__ __forceinline__ TileInfo tile_info(const FwdArgs &a, long long tile) {
    TileInfo t;
    const unsigned fu = (unsigned)tile;
    t.seq = (int)a.plan.divN.div(fu);
    t.n = (int)(fu - (unsigned)t.seq * (unsigned)a.plan.N);
    t.b = (int)a.divH.div((unsigned)t.seq);
    t.h = t.seq - t.b * a.heads;
    t.ntok = min(NT, a.T - t.n * NT);
    t.tok0 = ((size_t)t.b * a.T + (size_t)t.n * NT) * a.heads + t.h;
    return t;
}

// Products of the issuing thread: 8 k-steps of 16 each, unrolled with immediate descriptor offsets: every instruction
// of the issuing thread takes of the order of ten cycles beside the working warps of its scheduler, and the issue then
// keeps up with the tensor pipe (one tcgen05.mma per 64 to 78 cycles).
// D (+)= A x B with A (packed bf16 pairs, 8 columns per k-step of 16) in TMEM and B in shared memory
template <int ACC, uint32_t B_CONST>
__device__ __forceinline__ void mma_ts_c(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_base, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .b64 db;\n\t.reg .b32 lb;\n\t"
        "add.u32 lb, %2, %5;\n\tmov.b64 db, {lb, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, %6;\n\t}" ::"r"(d_tmem), "r"(a_tmem), "r"(b_base), "r"(idesc),
        "r"(kDescHi), "n"(B_CONST), "n"(ACC)
        : "memory");
}
// A = operand tile in TMEM (64 columns: channels 2 u, 2 u + 1 of a token in column u), B K-major
template <int ACC0, int NK = 8, int KS = 0>
__device__ __forceinline__ void mma8_ek(uint32_t d, uint32_t e_tmem, uint32_t b_base, uint32_t idesc) {
    if constexpr (KS < NK) {
        mma_ts_c<(KS == 0 ? ACC0 : 1), t_kmaj(0) + t_kstep(KS)>(d, e_tmem + 8 * KS, b_base, idesc);
        mma8_ek<ACC0, NK, KS + 1>(d, e_tmem, b_base, idesc);
    }
}
// The contractions over the channels: with head dimension 64 (zero-extended on chip) the channels 64..127 of every
// operand are zero, and the four k-steps over them are left out.
template <int ACC0>
__device__ __forceinline__ void prod_ek(bool half, uint32_t d, uint32_t e_tmem, uint32_t b_base) {
    if (half) mma8_ek<ACC0, 4>(d, e_tmem, b_base, kIdescKK);
    else mma8_ek<ACC0, 8>(d, e_tmem, b_base, kIdescKK);
}
template <int ACC0>
__device__ __forceinline__ void prod_kk(bool half, uint32_t d, uint32_t a_base, uint32_t b_base) {
    if (half) mma8_kk<ACC0, 4>(d, a_base, b_base, kIdescKK);
    else mma8_kk<ACC0, 8>(d, a_base, b_base, kIdescKK);
}
// The products of one request.  kb, hb, cb: descriptor bases (shared address >> 4) of the slot's buffers.
__device__ __forceinline__ void issue_batch(int op, bool half, uint32_t kb, uint32_t hb, uint32_t cb, uint32_t tm_S, uint32_t tm_R,
                                            uint32_t tm_E, uint32_t bar_s, uint32_t bar_r, uint32_t bar_sc) {
    switch (op) {
        case OP_FROB:    // Gram matrix Khat Khat^T and Khat H_0
            prod_kk<0>(half, tm_S, kb, kb);
            prod_kk<0>(half, tm_R, kb, hb);
            mma_commit(bar_s);
            break;
        case OP_ITER1:   // S = E Khat^T, R += E H_0^T (the second runs under the masked-score epilogue)
            prod_ek<0>(half, tm_S, tm_E, kb);
            mma_commit(bar_sc);
            if (half) mma_commit(bar_s);     // (the slot's compute warps take part in the masked-score epilogue)
            prod_ek<1>(half, tm_R, tm_E, hb);
            break;
        case OP_ITER2:   // R += P Khat
            mma8_pm_rows(tm_R, tm_S, kb, kIdescPM);
            mma_commit(bar_r);
            break;
        case OP_OUT_S:   // scores of the final iterate: S = X_hi Khat^T + X_lo Khat^T (X_lo sits in the first columns of R)
            prod_ek<0>(half, tm_S, tm_E, kb);
            prod_ek<1>(half, tm_S, tm_R, kb);
            mma_commit(bar_sc);
            prod_ek<0>(half, tm_R, tm_E, hb);   // O = X_hi U_0^T (runs under the masked-score epilogue; X_lo has been read)
            break;
        case OP_OUT_O:   // O += P V
            mma8_pm(tm_R, tm_S, cb, kIdescPM);
            mma_commit(bar_r);
            break;
        default:
            break;
    }
}

struct Ctx {
    int l, q, c;                  // lane, TMEM lane quadrant, token / TMEM lane of the slot's tile
    uint32_t tm_s, tm_r, tm_e;    // TMEM addresses of this thread's lane: scores, accumulator, operand
};

// Masked scores of 16 keys: S (fp32, 16 columns) -> P (packed bf16 pairs in 8 registers).  EXACT: per-element factor
// 2^(ac_c - G_j) (strongly decaying tiles, whose keys are not pre-scaled); KEYF: key j's column times ks[j] (the pass
// whose P meets the unscaled V); DIAG: keys i <= l of the 32-key block are visible (i0: first key of this half).
template <bool EXACT, bool KEYF, bool DIAG>
__device__ __forceinline__ void p_half(const uint32_t (&r)[16], uint32_t (&pk)[8], const float *G2h, const float *ksh,
                                       float ac_c, int l, int i0) {
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        float p0 = __uint_as_float(r[2 * u]), p1 = __uint_as_float(r[2 * u + 1]);
        if (EXACT) {
            p0 *= ex2_fast(fminf(ac_c - G2h[2 * u], 126.f));
            p1 *= ex2_fast(fminf(ac_c - G2h[2 * u + 1], 126.f));
        }
        if (KEYF) {
            const float2 f = *reinterpret_cast<const float2 *>(ksh + 2 * u);
            p0 *= f.x;
            p1 *= f.y;
        }
        if (DIAG) {
            p0 = (i0 + 2 * u <= l) ? p0 : 0.f;
            p1 = (i0 + 2 * u + 1 <= l) ? p1 : 0.f;
        }
        pk[u] = pack_bf16(p0, p1);
    }
}
// Masked-score epilogue of token c = 32 q + l: key blocks below q need no mask, block q is the diagonal block, the
// blocks above it are zero.  P for keys 32 kb + 2 u, 2 u + 1 goes to column 32 kb + u of the score tile.  The epilogue
// is a chain of tensor-memory round trips (loads of a 32-key block, conversion, stores), so the zero blocks are stored
// first.
template <bool EXACT, bool KEYF>
__device__ __forceinline__ void p_convert(const Ctx &cx, const GateScalars *gs, float ac_c, int kb, const uint32_t (&ra)[16],
                                          const uint32_t (&rb)[16]) {
    uint32_t pa[8], pb[8];
    const float *G2kb = gs->G2 + 32 * kb, *kskb = gs->ks + 32 * kb;
    if (kb == cx.q) {
        p_half<EXACT, KEYF, true>(ra, pa, G2kb, kskb, ac_c, cx.l, 0);
        p_half<EXACT, KEYF, true>(rb, pb, G2kb + 16, kskb + 16, ac_c, cx.l, 16);
    } else {
        p_half<EXACT, KEYF, false>(ra, pa, G2kb, kskb, ac_c, cx.l, 0);
        p_half<EXACT, KEYF, false>(rb, pb, G2kb + 16, kskb + 16, ac_c, cx.l, 16);
    }
    TMEM_ST8(cx.tm_s + 32 * kb, pa);
    TMEM_ST8(cx.tm_s + 32 * kb + 8, pb);
}
// Head dimension 64: key blocks of the masked scores that a token's score warp converts in an iteration; the token's
// compute warp, which has nothing else to do until the product that consumes the masked scores is complete, converts
// the rest.
__device__ __forceinline__ int p_split(int q) { return (q + 2) >> 1; }
// The masked-score epilogue of an iteration for the key blocks kb0 <= kb < kb1 of this thread's token.
template <bool EXACT>
__device__ __forceinline__ void p_epilogue_blocks(const Ctx &cx, const GateScalars *gs, float ac_c, int kb0, int kb1) {
#pragma unroll 1
    for (int kb = kb0; kb < kb1; ++kb) {
        uint32_t ra[16], rb[16];
        TMEM_LD16(cx.tm_s + 32 * kb, ra);
        TMEM_LD16(cx.tm_s + 32 * kb + 16, rb);
        tmem_wait_ld();
        p_convert<EXACT, false>(cx, gs, ac_c, kb, ra, rb);
    }
    tmem_wait_st();
}
template <bool EXACT, bool KEYF, bool SPLIT>
__device__ __forceinline__ void p_epilogue_t(const Ctx &cx, const GateScalars *gs, float ac_c) {
    if (!KEYF && SPLIT) {     // an iteration: the upper key blocks are left to the token's compute warp
        p_epilogue_blocks<EXACT>(cx, gs, ac_c, 0, p_split(cx.q));
        return;
    }
    if (KEYF) {      // (the product of an iteration leaves out the rows whose key block is above the diagonal instead)
        uint32_t z[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) z[i] = 0u;
#pragma unroll 1
        for (int kb = cx.q + 1; kb < 4; ++kb) {
            TMEM_ST8(cx.tm_s + 32 * kb, z);
            TMEM_ST8(cx.tm_s + 32 * kb + 8, z);
        }
    }
#pragma unroll 1
    for (int kb = 0; kb <= cx.q; ++kb) {
        uint32_t ra[16], rb[16];
        TMEM_LD16(cx.tm_s + 32 * kb, ra);
        TMEM_LD16(cx.tm_s + 32 * kb + 16, rb);
        tmem_wait_ld();
        p_convert<EXACT, KEYF>(cx, gs, ac_c, kb, ra, rb);
    }
    tmem_wait_st();
}
template <bool KEYF, bool SPLIT>
__device__ __forceinline__ void p_epilogue(const Ctx &cx, const GateScalars *gs, bool exact, float ac_c) {
    if (exact) p_epilogue_t<true, KEYF, SPLIT>(cx, gs, ac_c);
    else p_epilogue_t<false, KEYF, SPLIT>(cx, gs, ac_c);
}

// Sum over one 32-key block of the squared Gram entries of the earlier keys (decayed when the keys are not
// pre-scaled) and the key's own squared norm.
template <bool DIAG, bool EXACT>
__device__ __forceinline__ void gram_block(const uint32_t (&r)[32], const float *G2kb, float G2j, int l, float &gsum) {
    float acc[4] = {0.f, 0.f, 0.f, 0.f}, gd = 0.f;      // four partial sums: the additions do not wait for one another
#pragma unroll
    for (int ii = 0; ii < 32; ++ii) {
        const float g = __uint_as_float(r[ii]);
        const float g2 = g * g;
        if (DIAG) gd = ii == l ? g2 : gd;
        float w = EXACT ? ex2_fast(G2j - G2kb[ii]) * g2 : g2;
        if (DIAG) w = ii < l ? w : 0.f;
        acc[ii & 3] += w;
    }
    gsum += 2.f * ((acc[0] + acc[1]) + (acc[2] + acc[3])) + gd;
}

// Inclusive scan over the tile's 128 tokens (the slot's four warps, one token per thread) of the affine maps
// s -> a s + b, composed in token order; returns the map's value at `seed`.
__device__ __forceinline__ float affine_scan(const Ctx &cx, SlotScalars *sc, int slot, float a, float b, float seed) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float pa = __shfl_up_sync(0xffffffffu, a, o), pb = __shfl_up_sync(0xffffffffu, b, o);
        if (cx.l >= o) {
            b = fmaf(a, pb, b);
            a *= pa;
        }
    }
    // (the previous tile's carries have long been read: every warp of the slot has passed several hand-overs since)
    if (cx.l == 31) {
        sc->carry[0][cx.q] = a;
        sc->carry[1][cx.q] = b;
    }
    asm volatile("bar.sync %0, 128;" ::"r"(slot + 1) : "memory");
    float s = seed;
    for (int w = 0; w < cx.q; ++w) s = fmaf(sc->carry[0][w], s, sc->carry[1][w]);
    return fmaf(a, s, b);
}

template <bool EXTRA, bool HALF>
__global__ void __launch_bounds__(kThreadsSolve, 1)
fwd_tc_solve_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmO,
                    const __grid_constant__ CUtensorMap tmS, FwdArgs a, long long ntiles) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_bars[B_COUNT];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ __align__(16) uint32_t s_req[4];     // per slot: requests posted (warps), Gram matrices read (warps)
    __shared__ uint32_t s_sinfo[2];                 // score event n (parity): slot | read pass << 1 | gate buffer << 2 | (n + 1) << 8

    unsigned char *smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    const int tid = threadIdx.x;
    const uint32_t bars = smem_u32(&s_bars[0]);
    const uint32_t abort_addr = smem_u32(&s_abort);

    if (tid == 0) {
        s_abort = 0;
        s_req[0] = s_req[1] = s_req[2] = s_req[3] = 0u;
        s_sinfo[0] = s_sinfo[1] = 0u;
        for (int i = 0; i < B_COUNT; ++i) {
            const int b = i % B_PER_SLOT;
            const bool per_warp = i < B_DRAIN && (b == B_RDY_ST || b == B_QF || b == B_GF0 || b == B_GF1);
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bars + 8 * i), "r"(per_warp ? ST / 32 : 1));
        }
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
    const uint32_t sbase = smem_u32(smem);

    // this block's tiles: a contiguous range, dealt to the two slots in turn
    const long long t_lo = (ntiles * blockIdx.x) / gridDim.x, t_hi = (ntiles * (blockIdx.x + 1)) / gridDim.x;
    const int n_mine = (int)(t_hi - t_lo);
    const bool solve_only = EXTRA && a.solve_only != 0;   // the result is the solve itself: no V, no U, no output product
    const float *const beta_p = EXTRA ? a.beta : nullptr;
    const float *const alpha_p = EXTRA ? a.alpha : nullptr;
    const bool mix = alpha_p != nullptr && !solve_only;   // alpha-connection: the read uses alpha x + (1 - alpha) q
    // Head dimension 64: the slot's compute warps, idle while the slot has the score tile, convert the upper key blocks of
    // the masked scores of an iteration (with 128 channels this measured slower: the warps come later to their update)
    constexpr bool SPLIT = HALF;
    constexpr bool half = HALF;                           // head dimension 64: channels 64..127 are zero, their k-steps are left out

    // The helper warps come first: when a scheduler changes warps it prefers the oldest eligible one, and the thread
    // that issues the products must not wait behind the compute warps of its scheduler.
    if (tid < 128) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsHelper));
        const int hw = tid >> 5, lane = tid & 31;
        if (hw == 0) {
            // ================= gate scalars of every tile, one tile ahead of the compute warps =================
            for (int k = 0; k < n_mine; ++k) {
                const int slot = k & 1, j = k >> 1;
                const uint32_t sb = bars + 8 * (slot * B_PER_SLOT);
                if (j >= 2) wait_bar(sb + 8 * (B_GF0 + (j & 1)), (uint32_t)(((j - 2) >> 1) & 1), abort_addr);
                const TileInfo ti = tile_info(a, t_lo + k);
                GateScalars *g = &reinterpret_cast<SlotScalars *>(smem + OFF_SC + slot * SC_BYTES)->g[j & 1];
                float run = 0.f;
                float ks_g[4], ks_s[4];
#pragma unroll
                for (int grp = 0; grp < 4; ++grp) {
                    const int cc = 32 * grp + lane;
                    const bool in = cc < ti.ntok;       // tokens past the sequence: no decay, unit lambda / strengths
                    const size_t idx = ti.tok0 + (size_t)cc * a.heads;
                    const float gv = in ? __ldg(a.gate + idx) : 1.f;
                    const float lamv = in ? __ldg(a.lam + idx) : 1.f;
                    const float bv = (beta_p && in) ? __ldg(beta_p + idx) : 1.f;
                    const float av = (alpha_p && in) ? __ldg(alpha_p + idx) : 1.f;
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
                    g->al[cc] = av;
                    ks_g[grp] = G2c;
                    ks_s[grp] = sqrtf(fmaxf(bv, 0.f));
                }
                {
                    // the decay of the whole tile decides how the keys are staged (ti.ntok - 1 is the last token)
                    const float Glast = __shfl_sync(0xffffffffu, ks_g[(ti.ntok - 1) >> 5], (ti.ntok - 1) & 31);
                    const bool exact = Glast < -60.f;
#pragma unroll
                    for (int grp = 0; grp < 4; ++grp)
                        g->ks[32 * grp + lane] = exact ? ks_s[grp] : ks_s[grp] * exp2f(-0.5f * ks_g[grp]);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(sb + 8 * (B_GS0 + (j & 1)));
            }
        } else if (hw == 1 || hw == 3) {
            // ========== TMA thread of a slot: first loads, V once q has been read, result stores, the next q ==========
            const int slot = hw >> 1;
            const int n_slot = (n_mine - slot + 1) >> 1;       // tiles of this slot: k = slot, slot + 2, ...
            if (lane == 0 && n_slot > 0) {
                const uint32_t sb = bars + 8 * (slot * B_PER_SLOT);
                const uint32_t sl = sbase + slot * SLOT_BYTES;
                auto load_q = [&](int k) {
                    const TileInfo ti = tile_info(a, t_lo + k);
                    mbar_expect_tx(sb + 8 * B_LD_Q, 32768u);
                    tma_load_tile3(&tmQ, sl + BUF_C, sb + 8 * B_LD_Q, ti.h * a.d, tile_x_hi(ti.h, a.d, a.heads), ti.n * NT, ti.b);
                };
                // the inputs do not depend on the state kernel; its per-tile states do
                {
                    const TileInfo ti = tile_info(a, t_lo + slot);
                    load_q(slot);
                    mbar_expect_tx(sb + 8 * B_LD_K, 32768u);
                    tma_load_tile3(&tmK, sl + BUF_A, sb + 8 * B_LD_K, ti.h * a.d, tile_x_hi(ti.h, a.d, a.heads), ti.n * NT, ti.b);
                    asm volatile("griddepcontrol.wait;" ::: "memory");
                    mbar_expect_tx(sb + 8 * B_LD_H, 32768u);
                    tma_load_tile2(&tmS, sl + BUF_B, sb + 8 * B_LD_H, (int)((t_lo + slot) * 256));
                }
                for (int j = 0; j < n_slot; ++j) {
                    const int k = slot + 2 * j;
                    const TileInfo ti = tile_info(a, t_lo + k);
                    if (!solve_only) {
                        wait_bar(sb + 8 * B_QF, (uint32_t)(j & 1), abort_addr);
                        mbar_expect_tx(sb + 8 * B_LD_V, 32768u);
                        tma_load_tile3(&tmV, sl + BUF_C, sb + 8 * B_LD_V, ti.h * a.d, tile_x_hi(ti.h, a.d, a.heads), ti.n * NT, ti.b);
                    }
                    wait_bar(sb + 8 * B_RDY_ST, (uint32_t)(j & 1), abort_addr);
                    for (int hf = 0; hf < a.d / 64; ++hf)   // rows past the sequence are clipped; channels from a.d on are not stored
                        asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];" ::
                                         "l"(reinterpret_cast<uint64_t>(&tmO)), "r"(ti.h * a.d + 64 * hf), "r"(ti.n * NT),
                                     "r"(ti.b), "r"(sl + BUF_C + 16384 * hf)
                                     : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the staged tile has been read
                    if (j + 1 < n_slot && !aborted(abort_addr)) load_q(k + 2);
                }
                asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // output stores are complete
            }
        } else {
            // ================================ MMA issuing thread ================================
            // Serves the requests of both slots in the order they become ready.  The score tile S is held by a slot
            // from its FROB request until its warps have read the Gram matrix (counted in shared memory), from ITER1 to the issue of
            // ITER2 and from OUT_S to the issue of OUT_O (products run in issue order, so the next owner's score
            // product follows the last read of P).
            if (lane == 0) {
                const uint32_t base14 = (sbase >> 4) & 0x3FFF;
                // Per-slot state in scalars (arrays indexed by the slot would live in local memory).  Every instruction
                // of this thread competes with the compute warps of its scheduler, so the paths between a request and
                // its products are kept as short as possible.
                int op0 = OP_FROB, op1 = OP_FROB, it0 = 0, it1 = 0, left0 = (n_mine + 1) >> 1, left1 = n_mine >> 1;
                uint32_t thr0 = 4u, thr1 = 4u;          // request counter values at which the next request of a slot is complete
                uint32_t gthr0 = 4u, gthr1 = 4u;        // the same for the Gram-read counters
                uint32_t til0 = 0, til1 = 0;            // tiles done (phase of the per-tile TMA barriers)
                const uint32_t req_addr = smem_u32(&s_req[0]);
                int owner = -1;                         // slot that holds S while its warps read the Gram matrix
                int prefer = 0;                         // slot to serve first when both are ready
                bool gave_up = false;
                uint32_t sev = 0;                       // score events so far
                const uint32_t sinfo_addr = smem_u32(&s_sinfo[0]);
                auto issue = [&](int sl, int o) {
                    const uint32_t sbb = bars + 8 * (sl * B_PER_SLOT);
                    const uint32_t sl14 = base14 + ((sl * SLOT_BYTES) >> 4);
                    if (o == OP_ITER1 || o == OP_OUT_S) {   // tell the score warps whose scores come next
                        ++sev;
                        const uint32_t info = (uint32_t)sl | (o == OP_OUT_S ? 2u : 0u) | (((sl ? til1 : til0) & 1u) << 2) | (sev << 8);
                        asm volatile("st.volatile.shared::cta.u32 [%0], %1;" ::"r"(sinfo_addr + 4u * ((sev - 1u) & 1u)), "r"(info) : "memory");
                    }
                    fence_after();
                    issue_batch(o, half, sl14 + (BUF_A >> 4), sl14 + (BUF_B >> 4), sl14 + (BUF_C >> 4), tmem + TM_S, tmem + tm_r_of(sl),
                                tmem + tm_e_of(sl), sbb + 8 * B_MMA_S, sbb + 8 * B_MMA_R, bars + 8 * B_SC);
                };
                // Bookkeeping of a request of slot sl that has just been issued, together with its follow-up (ITER2 after
                // ITER1, OUT_O after OUT_S): the slot's next request, counters and tile count.  Returns the counter value
                // at which the follow-up is posted.
                auto book = [&](int sl, int o) -> uint32_t {
                    bool tile_done = false;
                    int it = sl ? it1 : it0, nop;
                    // (the masked scores of an iteration come from the score warps and the slot's compute warps)
                    const uint32_t thr = (sl ? thr1 : thr0) + (SPLIT && o == OP_ITER1 ? 8u : 4u);
                    if (o == OP_FROB) {
                        owner = sl;                          // until the Gram matrix has been read
                        nop = it < a.n_iter ? OP_ITER1 : OP_OUT_S;
                        if (a.n_iter == 0 && solve_only) tile_done = true;
                    } else if (o == OP_ITER1) {
                        ++it;
                        nop = it < a.n_iter ? OP_ITER1 : OP_OUT_S;
                        if (it >= a.n_iter && solve_only) tile_done = true;
                    } else {
                        nop = OP_FROB;
                        tile_done = true;
                    }
                    if (tile_done) {
                        nop = OP_FROB;
                        it = 0;
                    }
                    if (sl) { op1 = nop; it1 = it; thr1 = thr + (o == OP_FROB ? 0u : 4u); if (tile_done) { --left1; ++til1; } }
                    else { op0 = nop; it0 = it; thr0 = thr + (o == OP_FROB ? 0u : 4u); if (tile_done) { --left0; ++til0; } }
                    return thr;
                };
                int next_s = -1;                        // slot known to have its request posted (no poll needed)
                while ((left0 > 0 || left1 > 0) && !gave_up) {
                    // ---- a slot whose next request (FROB, ITER1 or OUT_S: all need the score tile) is posted and may have S
                    int s = next_s;
                    next_s = -1;
                    for (int polls = 0; s < 0;) {
                        uint32_t c0, c1, g0, g1;
                        asm volatile("ld.volatile.shared::cta.v4.u32 {%0, %1, %2, %3}, [%4];"
                                     : "=r"(c0), "=r"(c1), "=r"(g0), "=r"(g1)
                                     : "r"(req_addr)
                                     : "memory");
                        if (owner == 0 && (int)(g0 - gthr0) >= 0) { gthr0 += 4u; owner = -1; }
                        if (owner == 1 && (int)(g1 - gthr1) >= 0) { gthr1 += 4u; owner = -1; }
                        const bool r0 = left0 > 0 && owner != 1 && (int)(c0 - thr0) >= 0;
                        const bool r1 = left1 > 0 && owner != 0 && (int)(c1 - thr1) >= 0;
                        if (r0 | r1) {
                            s = (r0 && !(r1 && prefer == 1)) ? 0 : 1;
                            break;
                        }
                        if ((++polls & 1023) == 0 && (aborted(abort_addr) || polls > (1 << 24))) {
                            gave_up = true;
                            break;
                        }
                    }
                    if (gave_up) break;
                    prefer = 1 - s;
                    int o = s ? op1 : op0;
                    // a request of the slot that still holds S for its Gram reads implies that those are done
                    if (owner == s) {
                        if (s) gthr1 += 4u; else gthr0 += 4u;
                        owner = -1;
                    }
                    uint32_t til = s ? til1 : til0;
                    if (o == OP_FROB) wait_bar(bars + 8 * (s * B_PER_SLOT + B_LD_H), til & 1u, abort_addr);   // the H_0 tile (TMA)
                    if (o == OP_OUT_S) wait_bar(bars + 8 * (s * B_PER_SLOT + B_LD_U), til & 1u, abort_addr);  // the U_0 tile
                    issue(s, o);
                    uint32_t thr = book(s, o);
                    if (o == OP_FROB) continue;
                    // ---- ITER1 or OUT_S of slot s is running: its follow-up (ITER2, OUT_O) comes next.  In the steady state
                    // of the iterations the other slot's ITER1 follows at once; everything both need is worked out here,
                    // while the products run and the score warps work, so that a handful of instructions lie between the
                    // posts and the products.
                    for (;;) {
                        const int t = 1 - s;
                        const uint32_t s14 = base14 + ((s * SLOT_BYTES) >> 4), t14 = base14 + ((t * SLOT_BYTES) >> 4);
                        const uint32_t p_kb = s14 + (BUF_A >> 4), p_tmR = tmem + tm_r_of(s);
                        const uint32_t p_barR = bars + 8 * (s * B_PER_SLOT + B_MMA_R);
                        const bool t_iter = (t ? left1 : left0) > 0 && (t ? op1 : op0) == OP_ITER1;
                        const uint32_t thr_t = t ? thr1 : thr0;
                        const uint32_t n_kb = t14 + (BUF_A >> 4), n_tmE = tmem + tm_e_of(t);
                        const uint32_t n_barS = bars + 8 * (t * B_PER_SLOT + B_MMA_S);
                        const uint32_t n_info = (uint32_t)t | (((t ? til1 : til0) & 1u) << 2) | ((sev + 1u) << 8);
                        const uint32_t n_sinfo = sinfo_addr + 4u * (sev & 1u);
                        uint32_t c_t = 0u;
                        for (int polls = 0;;) {
                            uint32_t c0, c1;
                            asm volatile("ld.volatile.shared::cta.v2.u32 {%0, %1}, [%2];" : "=r"(c0), "=r"(c1) : "r"(req_addr) : "memory");
                            c_t = s ? c0 : c1;
                            if ((int)((s ? c1 : c0) - thr) >= 0) break;
                            if ((++polls & 1023) == 0 && (aborted(abort_addr) || polls > (1 << 24))) {
                                gave_up = true;
                                break;
                            }
                        }
                        if (gave_up) break;
                        if (o == OP_ITER1) {
                            fence_after();
                            mma8_pm_rows(p_tmR, tmem + TM_S, p_kb, kIdescPM);  // ITER2: R += P Khat
                            mma_commit(p_barR);
                        } else {                                 // OUT_O: the V tile (TMA)
                            wait_bar(bars + 8 * (s * B_PER_SLOT + B_LD_V), til & 1u, abort_addr);
                            issue(s, OP_OUT_O);
                        }
                        bool t_posted = (int)(c_t - thr_t) >= 0;
                        if (t_iter && !t_posted) {
                            // the other slot is in its iterations and its update is about to end (this slot's own next
                            // request is a whole update away): wait for it here, where its products are prepared
                            for (int polls = 0; polls < 4096 && !t_posted; ++polls) {
                                uint32_t c0, c1;
                                asm volatile("ld.volatile.shared::cta.v2.u32 {%0, %1}, [%2];" : "=r"(c0), "=r"(c1) : "r"(req_addr) : "memory");
                                t_posted = (int)((t ? c1 : c0) - thr_t) >= 0;
                            }
                        }
                        if (!(t_iter && t_posted)) {
                            // the other slot's request, if it was already posted, is served next without a poll
                            if ((t ? left1 : left0) > 0 && t_posted) next_s = t;
                            break;
                        }
                        // ---- ITER1 of the other slot, at once
                        asm volatile("st.volatile.shared::cta.u32 [%0], %1;" ::"r"(n_sinfo), "r"(n_info) : "memory");
                        ++sev;
                        fence_after();
                        prod_ek<0>(half, tmem + TM_S, n_tmE, n_kb);           // S = E Khat^T
                        mma_commit(bars + 8 * B_SC);
                        if (SPLIT) mma_commit(n_barS);
                        prod_ek<1>(half, tmem + tm_r_of(t), n_tmE, n_kb + ((BUF_B - BUF_A) >> 4));   // R += E H_0^T
                        if (owner == t) {                        // (its Gram reads are done: it has asked again)
                            if (t) gthr1 += 4u; else gthr0 += 4u;
                            owner = -1;
                        }
                        prefer = s;
                        til = t ? til1 : til0;
                        thr = book(t, OP_ITER1);
                        o = OP_ITER1;
                        s = t;
                    }
                }
                if (gave_up) set_abort(abort_addr);
                // every product is complete before the block gives its tensor memory back
                mma_commit(bars + 8 * B_DRAIN);
                if (!mbar_spin_bounded(bars + 8 * B_DRAIN, 0u)) set_abort(abort_addr);
            }
        }
    } else if (tid < 256) {
        // ================================== score warps ==================================
        // The masked-score epilogue of both slots: S (fp32) -> P (packed bf16) in place, for the scores of an iteration
        // and for those of the read.  These warps hold no iterate, so they are not short of registers, and the compute
        // warps go from their update straight to the wait for the accumulator.
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsScore));
        Ctx cx;
        cx.l = tid & 31;
        cx.q = (tid >> 5) & 3;
        cx.c = 32 * cx.q + cx.l;
        cx.tm_s = tmem + TM_S + ((uint32_t)(32 * cx.q) << 16);
        cx.tm_r = cx.tm_e = 0u;
        const int per_tile = a.n_iter + (solve_only ? 0 : 1);
        const long long n_events = (long long)n_mine * per_tile;
        int reads0 = 0, reads1 = 0;         // read passes seen per slot (= tiles done)
        for (long long ev = 0; ev < n_events; ++ev) {
            // The issuing thread announces an event before it issues the score product: whose scores, which pass; the
            // scalars the epilogue needs are fetched while the product runs.
            uint32_t info = 0u;
            if (cx.l == 0) {
                for (int polls = 0;; ++polls) {
                    asm volatile("ld.volatile.shared::cta.u32 %0, [%1];" : "=r"(info) : "r"(smem_u32(&s_sinfo[ev & 1])) : "memory");
                    if ((info >> 8) == (uint32_t)(ev + 1)) break;
                    if ((polls & 1023) == 1023 && (aborted(abort_addr) || polls > (1 << 24))) {
                        set_abort(abort_addr);
                        break;
                    }
                }
            }
            info = __shfl_sync(0xffffffffu, info, 0);
            const int sl_ = (int)(info & 1u);
            const SlotScalars *const scs = reinterpret_cast<const SlotScalars *>(smem + OFF_SC + sl_ * SC_BYTES);
            const GateScalars *const gs = &scs->g[(info >> 2) & 1u];
            const bool exact = scs->exact[(info >> 2) & 1u] != 0;
            const float ac_c = gs->ac[cx.c];
            wait_bar(bars + 8 * B_SC, (uint32_t)(ev & 1), abort_addr);
            fence_after();
            if (info & 2u) {
                // the score products of the read pass were the last readers of the slot's keys: the next tile's keys
                // are loaded now, and the slot's compute warps scale them while the read runs
                const int kdone = sl_ + kSlots * (sl_ ? reads1 : reads0);
                if (tid == 128 && kdone + kSlots < n_mine) {
                    const TileInfo tn = tile_info(a, t_lo + kdone + kSlots);
                    const uint32_t bar_k = bars + 8 * (sl_ * B_PER_SLOT + B_LD_K);
                    mbar_expect_tx(bar_k, 32768u);
                    tma_load_tile3(&tmK, sbase + sl_ * SLOT_BYTES + BUF_A, bar_k, tn.h * a.d, tile_x_hi(tn.h, a.d, a.heads), tn.n * NT, tn.b);
                }
                if (sl_) ++reads1; else ++reads0;
                p_epilogue<true, SPLIT>(cx, gs, exact, ac_c);
            } else {
                p_epilogue<false, SPLIT>(cx, gs, exact, ac_c);
            }
            fence_before();
            warp_post(smem_u32(&s_req[sl_]), cx.l);          // -> ITER2 / OUT_O of that slot
        }
    } else {
        // ================================= compute threads =================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsCompute));
        const int slot = (tid >> 7) - 2;
        Ctx cx;
        cx.l = tid & 31;
        cx.q = (tid >> 5) & 3;
        cx.c = 32 * cx.q + cx.l;
        const uint32_t lane_addr = (uint32_t)(32 * cx.q) << 16;
        cx.tm_s = tmem + TM_S + lane_addr;
        cx.tm_r = tmem + tm_r_of(slot) + lane_addr;
        cx.tm_e = tmem + tm_e_of(slot) + lane_addr;
        const int c = cx.c, l = cx.l;
        const bool leader = c == 0;                              // issues the slot's loads that follow a product
        const bool adaptive = (a.flags & GKA_FLAG_ADAPTIVE_LAMBDA) != 0;
        const uint32_t sb = bars + 8 * (slot * B_PER_SLOT);
        const uint32_t sl = sbase + slot * SLOT_BYTES;
        unsigned char *const bufa = smem + slot * SLOT_BYTES + BUF_A, *const bufc = smem + slot * SLOT_BYTES + BUF_C;
        SlotScalars *const sc = reinterpret_cast<SlotScalars *>(smem + OFF_SC + slot * SC_BYTES);
        // the per-tile states and norms come from the state kernel
        asm volatile("griddepcontrol.wait;" ::: "memory");

        // Head dimension 64: the passes over the channels stop at channel 64 (the rest is zero in every operand and stays so)
        constexpr int NG16 = HALF ? 4 : 8;    // groups of 16 channels
        uint64_t xs[64];                      // -zt_c x_c: the token's 128 channels as fp32 pairs
        uint32_t n_s = 0, n_r = 0;            // completed phases of MMA_S, MMA_R
        auto wait_s = [&]() { wait_bar(sb + 8 * B_MMA_S, n_s & 1u, abort_addr); ++n_s; fence_after(); };
        auto wait_r = [&]() { wait_bar(sb + 8 * B_MMA_R, n_r & 1u, abort_addr); ++n_r; fence_after(); };
        const uint32_t req_addr = smem_u32(&s_req[slot]), grd_addr = smem_u32(&s_req[2 + slot]);
        auto arrive_rdy = [&]() { warp_post(req_addr, l); };
        // -xs (times `scale`) as packed bf16 pairs of channel group g8 (8 channels): its leading part, or the remainder
        auto pack_x = [&](int g8, bool lo, float scale, uint32_t(&pk)[4]) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float xa, xb;
                f2_unpack(xs[4 * g8 + u], xa, xb);
                xa *= -scale;
                xb *= -scale;
                uint32_t p = pack_bf16(xa, xb);
                if (lo) p = pack_bf16(xa - bf16_lo(p), xb - bf16_hi(p));
                pk[u] = p;
            }
        };

        for (int k = slot, j = 0; k < n_mine; k += kSlots, ++j) {
            const long long tile = t_lo + k;
            const bool more = k + kSlots < n_mine;
            const GateScalars *const gs = &sc->g[j & 1];
            const TileInfo ti = tile_info(a, tile);
            const bool valid = c < ti.ntok;
            // loads of the slot's next tile, issued by the leader as soon as the buffer's last reader is done
            auto load_next_k = [&]() {
                if (leader && more) {
                    const TileInfo tn = tile_info(a, tile + kSlots);
                    mbar_expect_tx(sb + 8 * B_LD_K, 32768u);
                    tma_load_tile3(&tmK, sl + BUF_A, sb + 8 * B_LD_K, tn.h * a.d, tile_x_hi(tn.h, a.d, a.heads), tn.n * NT, tn.b);
                }
            };
            auto load_next_h = [&]() {
                if (leader && more) {
                    mbar_expect_tx(sb + 8 * B_LD_H, 32768u);
                    tma_load_tile2(&tmS, sl + BUF_B, sb + 8 * B_LD_H, (int)((tile + kSlots) * 256));
                }
            };
            auto after_last_h0_product = [&]() {      // H_0 has been read for the last time
                if (solve_only) {
                    load_next_k();
                    load_next_h();
                } else if (leader) {
                    mbar_expect_tx(sb + 8 * B_LD_U, 32768u);
                    tma_load_tile2(&tmS, sl + BUF_B, sb + 8 * B_LD_U, (int)(tile * 256 + 128));
                }
            };
            // ||H_0||_F^2 of the tile (state kernel): fetched now, used by the scan
            const float hh = ldg_stream_f32(a.tile_hh + tile);
            // ---- gate scalars (helper warp) and the K tile (TMA) of this tile
            // Khat of tile jj of this slot: gate scalars (helper warp) and K tile (TMA) awaited, the token's key row scaled
            // in place
            auto stage_keys = [&](int jj) {
                wait_bar(sb + 8 * (B_GS0 + (jj & 1)), (uint32_t)((jj >> 1) & 1), abort_addr);
                wait_bar(sb + 8 * B_LD_K, (uint32_t)(jj & 1), abort_addr);
                const float fj = sc->g[jj & 1].ks[c];
                const uint64_t f2 = f2_pack(fj, fj);
#pragma unroll 1
                for (int g = 0; g < 2 * NG16; ++g) {             // (rolled: code that runs once per tile is kept small)
                    uint4 v = *reinterpret_cast<const uint4 *>(bufa + tile_off(c, g));
                    uint32_t *pv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        float lo, hi;
                        f2_unpack(f2_mul(f2_pack(bf16_lo(pv[u]), bf16_hi(pv[u])), f2), lo, hi);
                        pv[u] = pack_bf16(lo, hi);
                    }
                    *reinterpret_cast<uint4 *>(bufa + tile_off(c, g)) = v;
                }
                fence_async_smem();
            };
            if (j == 0 || solve_only) stage_keys(j);             // (otherwise done under the previous tile's read)
            const bool exact = gs->G2[ti.ntok - 1] < -60.f;     // the tile decays below 2^-60: per-element factors
            if (leader) sc->exact[j & 1] = exact ? 1 : 0;       // (for the score warps; published by the FROB request)
            const float G2c = gs->G2[c];
            arrive_rdy();                                        // -> FROB
            wait_s();
            if (a.n_iter == 0) after_last_h0_product();
            // ---- chunk-wise Frobenius norms: for the token's key, k^T H_0 k and the decayed squared Gram entries of
            // the earlier keys
            float kh = 0.f, gsum = 0.f;
            {
                float khp[4] = {0.f, 0.f, 0.f, 0.f};
                uint32_t ra[32];
                // (the Gram matrix first: it sits in the score tile, which the other slot is waiting for)
#pragma unroll 1
                for (int kb = 0; kb <= cx.q; ++kb) {
                    TMEM_LD32(cx.tm_s + 32 * kb, ra);
                    tmem_wait_ld();
                    if (exact) {
                        if (kb == cx.q) gram_block<true, true>(ra, gs->G2 + 32 * kb, G2c, l, gsum);
                        else gram_block<false, true>(ra, gs->G2 + 32 * kb, G2c, l, gsum);
                    } else {
                        if (kb == cx.q) gram_block<true, false>(ra, gs->G2 + 32 * kb, G2c, l, gsum);
                        else gram_block<false, false>(ra, gs->G2 + 32 * kb, G2c, l, gsum);
                    }
                }
                fence_before();
                warp_post(grd_addr, l);                          // the Gram matrix has been read: S is free again
#pragma unroll 1
                for (int p = 0; p < NG16 / 2; ++p) {
                    TMEM_LD32(cx.tm_r + 32 * p, ra);
                    uint4 kv[4];
#pragma unroll
                    for (int h4 = 0; h4 < 4; ++h4) kv[h4] = *reinterpret_cast<const uint4 *>(bufa + tile_off(c, 4 * p + h4));
                    tmem_wait_ld();
#pragma unroll
                    for (int h4 = 0; h4 < 4; ++h4) {
                        const uint32_t *pk = reinterpret_cast<const uint32_t *>(&kv[h4]);
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            khp[h4] = fmaf(__uint_as_float(ra[8 * h4 + 2 * u]), bf16_lo(pk[u]), khp[h4]);
                            khp[h4] = fmaf(__uint_as_float(ra[8 * h4 + 2 * u + 1]), bf16_hi(pk[u]), khp[h4]);
                        }
                    }
                }
                kh = (khp[0] + khp[1]) + (khp[2] + khp[3]);
            }
            // ---- f_c by an affine scan (s_c = gamma_c^2 s_{c-1} + d_c, s_{-1} = ||H_0||^2), Chebyshev set-up
            float rho2, czb, lz;
            {
                // pre-scaled keys: both sums carry 2^(-2 G_c); plain keys: k H_0 k carries zeta_c
                const float dc = exact ? fmaf(2.f * ex2_fast(G2c), kh, gsum) : ex2_fast(2.f * G2c) * fmaf(2.f, kh, gsum);
                const float s = affine_scan(cx, sc, slot, ex2_fast(2.f * gs->lg[c]), dc, hh);
                const float fc = sqrtf(fmaxf(s, 0.f));
                float lamc = gs->lam[c];
                if (adaptive) lamc *= fc;
                const float Lpm = fc + 2.f * lamc;
                const float iL = 1.f / Lpm;
                const float rho = fc * iL;
                rho2 = rho * rho;
                czb = valid ? -gs->zt[c] * (2.f * iL) : 0.f;
                lz = lamc * gs->iz[c];
                if (a.fro_out && valid) a.fro_out[ti.tok0 + (size_t)c * a.heads] = fc;
            }
            wait_bar(sb + 8 * B_LD_Q, (uint32_t)(j & 1), abort_addr);   // q tile has landed
            // ---- x_0: R = q, E_0 = czb q, xs = E_0
#pragma unroll
            for (int g16 = 0; g16 < NG16; ++g16) {
                uint32_t rr[16], pk[8];
#pragma unroll
                for (int h2 = 0; h2 < 2; ++h2) {
                    const uint4 qv = *reinterpret_cast<const uint4 *>(bufc + tile_off(c, 2 * g16 + h2));
                    const uint32_t *qq = reinterpret_cast<const uint32_t *>(&qv);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float qa = bf16_lo(qq[u]), qb = bf16_hi(qq[u]);
                        rr[8 * h2 + 2 * u] = __float_as_uint(qa);
                        rr[8 * h2 + 2 * u + 1] = __float_as_uint(qb);
                        const uint32_t p = pack_bf16(czb * qa, czb * qb);
                        pk[4 * h2 + u] = p;
                        xs[8 * g16 + 4 * h2 + u] = f2_pack(bf16_lo(p), bf16_hi(p));
                    }
                }
                TMEM_ST16(cx.tm_r + 16 * g16, rr);
                TMEM_ST8(cx.tm_e + 8 * g16, pk);
            }
            if (!solve_only && !mix) warp_arrive(sb + 8 * B_QF, l);      // q has been read: V may take its buffer
            tmem_wait_st();
            // ---- Algorithm 1
            float omega = 2.f;
            if (a.n_iter > 0) {
                fence_before();
                arrive_rdy();                                    // -> ITER1
            }
            for (int it = 0; it < a.n_iter; ++it) {
                const bool last = it + 1 == a.n_iter;
                omega = 4.f / (4.f - rho2 * omega);              // weight schedule
                const float beta = omega - 1.f, cz = czb * omega;
                const uint64_t beta2 = f2_pack(beta, beta), cz2 = f2_pack(cz, cz), lz2 = f2_pack(lz, lz);
                // this warp's share of the masked-score epilogue (the upper key blocks of its tokens)
                if (SPLIT) {
                    wait_s();
                    if (exact) p_epilogue_blocks<true>(cx, gs, gs->ac[c], p_split(cx.q), cx.q + 1);
                    else p_epilogue_blocks<false>(cx, gs, 0.f, p_split(cx.q), cx.q + 1);
                    fence_before();
                    arrive_rdy();                                // -> ITER2 (with the score warps' posts)
                }
                wait_r();
                if (last) after_last_h0_product();
                // e_new = beta e_old + cz (R + lz xs) as bf16, xs += e_new (the value the operand holds).  Sixteen
                // channels at a time; the next group's loads are in flight while a group is computed.
                {
                    uint32_t ra[16], rb[16], ea[8], eb[8];
                    TMEM_LD16(cx.tm_r, ra);
                    TMEM_LD8(cx.tm_e, ea);
                    tmem_wait_ld();
#pragma unroll
                    for (int g = 0; g < NG16; ++g) {
                        uint32_t(&r)[16] = (g & 1) ? rb : ra;
                        uint32_t(&rn)[16] = (g & 1) ? ra : rb;
                        uint32_t(&e)[8] = (g & 1) ? eb : ea;
                        uint32_t(&en_)[8] = (g & 1) ? ea : eb;
                        if (g < NG16 - 1) {
                            TMEM_LD16(cx.tm_r + 16 * (g + 1), rn);
                            TMEM_LD8(cx.tm_e + 8 * (g + 1), en_);
                        }
                        uint32_t pk[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const int i = 8 * g + u;
                            const uint64_t res = f2_fma(lz2, xs[i], f2_pack(__uint_as_float(r[2 * u]), __uint_as_float(r[2 * u + 1])));
                            const uint64_t en = f2_fma(cz2, res, f2_mul(beta2, f2_pack(bf16_lo(e[u]), bf16_hi(e[u]))));
                            float ea_, eb_;
                            f2_unpack(en, ea_, eb_);
                            pk[u] = pack_bf16(ea_, eb_);
                            xs[i] = f2_add(xs[i], f2_pack(bf16_lo(pk[u]), bf16_hi(pk[u])));
                        }
                        TMEM_ST8(cx.tm_e + 8 * g, pk);
                                        if (g < NG16 - 1) tmem_wait_ld();
                    }
                    if (!last) {
                        tmem_wait_st();
                        fence_before();
                        arrive_rdy();                            // -> ITER1
                    }
                }
            }
            // ---- final iterate
            if (solve_only) {
                // the solve is the result: x_c = -xs / zt_c as bf16, staged in the q buffer and stored by TMA
                const float izc = gs->iz[c];
#pragma unroll
                for (int g8 = 0; g8 < 2 * NG16; ++g8) {
                    uint32_t pk[4];
                    pack_x(g8, false, izc, pk);
                    *reinterpret_cast<uint4 *>(bufc + tile_off(c, g8)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
                fence_async_smem();
                warp_arrive(sb + 8 * (B_GF0 + (j & 1)), l);
                warp_arrive(sb + 8 * B_RDY_ST, l);
                continue;
            }
            if (mix) {
                // alpha-connection (Section 4.3): the read uses alpha x + (1 - alpha) q; q is still in its buffer
                const float alc = gs->al[c], nzt = valid ? -gs->zt[c] : 0.f;
#pragma unroll
                for (int g8 = 0; g8 < 2 * NG16; ++g8) {
                    const uint4 qv = *reinterpret_cast<const uint4 *>(bufc + tile_off(c, g8));
                    const uint32_t *qq = reinterpret_cast<const uint32_t *>(&qv);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        float xa, xb;
                        f2_unpack(xs[4 * g8 + u], xa, xb);
                        const float qa = nzt * bf16_lo(qq[u]), qb = nzt * bf16_hi(qq[u]);
                        xs[4 * g8 + u] = f2_pack(fmaf(alc, xa - qa, qa), fmaf(alc, xb - qb, qb));
                    }
                }
                warp_arrive(sb + 8 * B_QF, l);                   // q has been read: V may take its buffer
            }
            // The read uses the final iterate as two bf16 terms in the score product (the recent keys resolve directions
            // of x that one bf16 rounding would lose): the leading term takes the operand columns, the remainder the
            // first columns of the accumulator, whose content is no longer needed.
#pragma unroll
            for (int g8 = 0; g8 < 2 * NG16; g8 += 2) {
                uint32_t hi[8], lo[8];
                pack_x(g8, false, 1.f, *reinterpret_cast<uint32_t(*)[4]>(&hi[0]));
                pack_x(g8 + 1, false, 1.f, *reinterpret_cast<uint32_t(*)[4]>(&hi[4]));
                pack_x(g8, true, 1.f, *reinterpret_cast<uint32_t(*)[4]>(&lo[0]));
                pack_x(g8 + 1, true, 1.f, *reinterpret_cast<uint32_t(*)[4]>(&lo[4]));
                TMEM_ST8(cx.tm_e + 4 * g8, hi);
                TMEM_ST8(cx.tm_r + 4 * g8, lo);
            }
            tmem_wait_st();
            fence_before();
            arrive_rdy();                                        // -> OUT_S
            // (the score warps mask the scores and post OUT_O; the values stay as loaded: their row factor
            // sqrt(beta_j) 2^(-G_j / 2) rides on the masked scores)
            if (more) stage_keys(j + 1);                         // the next tile's keys (loaded by a score warp at the read pass)
            wait_r();
            load_next_h();                                       // every product of the tile is complete
            // O as bf16 into the V buffer (no product reads it any more), stored by TMA
            {
                // (the iterate's registers are free by now: all four loads are in flight at once)
                uint32_t r[4][32];
#pragma unroll
                for (int p = 0; p < NG16 / 2; ++p) TMEM_LD32(cx.tm_r + 32 * p, r[p]);
                tmem_wait_ld();
#pragma unroll
                for (int p = 0; p < NG16 / 2; ++p) {
#pragma unroll
                    for (int h4 = 0; h4 < 4; ++h4) {
                        uint32_t pk[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) pk[u] = pack_bf16(__uint_as_float(r[p][8 * h4 + 2 * u]), __uint_as_float(r[p][8 * h4 + 2 * u + 1]));
                        *reinterpret_cast<uint4 *>(bufc + tile_off(c, 4 * p + h4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
            }
            fence_async_smem();
            fence_before();
            warp_arrive(sb + 8 * (B_GF0 + (j & 1)), l);
            warp_arrive(sb + 8 * B_RDY_ST, l);
        }
    }

    fence_before();
    __syncthreads();
    if (s_abort != 0) {
        // a wait gave up: leave time for copies still in flight before the shared memory is given back
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        if (tid == 0 && a.device_status) atomicExch(a.device_status, (int)GKA_ERR_TIMEOUT);
    }
    if (tid < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
}

}  // namespace

cudaError_t launch_fwd_solve(const FwdArgs &a, cudaStream_t stream) {
    alignas(64) CUtensorMap tmK, tmV, tmQ, tmO, tmS;
    const int cols = a.heads * a.d;
    const long long ntiles = a.plan.NC;
    if (!make_tile_map(&tmK, a.k, a.B, a.T, cols, NT) || !make_tile_map(&tmV, a.v, a.B, a.T, cols, NT) ||
        !make_tile_map(&tmQ, a.q, a.B, a.T, cols, NT) || !make_tile_map(&tmO, a.out, a.B, a.T, cols, NT) ||
        !make_state_map(&tmS, a.tile_hu, (unsigned long long)ntiles * 256ull))
        return cudaErrorInvalidValue;
    const bool extra = a.beta != nullptr || a.alpha != nullptr || a.solve_only != 0;
    const bool half = a.d == 64;
    auto kernel = extra ? (half ? fwd_tc_solve_kernel<true, true> : fwd_tc_solve_kernel<true, false>)
                        : (half ? fwd_tc_solve_kernel<false, true> : fwd_tc_solve_kernel<false, false>);
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SOLVE_SMEM);
    if (err != cudaSuccess) return err;
    int dev = 0, sms = 0;
    if ((err = cudaGetDevice(&dev)) != cudaSuccess) return err;
    if ((err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return err;
    const long long want = ntiles < sms ? ntiles : (long long)sms;   // one persistent block per SM, two tiles in flight each
    if (a.ev_start) cudaEventRecord(a.ev_start, stream);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(want < 1 ? 1 : want));
    cfg.blockDim = dim3(kThreadsSolve);
    cfg.dynamicSmemBytes = SOLVE_SMEM;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.ev_start ? 0 : 1;
    err = cudaLaunchKernelEx(&cfg, kernel, tmK, tmV, tmQ, tmO, tmS, a, ntiles);
    if (err != cudaSuccess) return err;
    if (a.ev_stop) cudaEventRecord(a.ev_stop, stream);
    return cudaGetLastError();
}

}  // namespace gka
