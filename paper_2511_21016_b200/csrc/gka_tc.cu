// tcgen05 / TMEM chunk-wise GKA forward (bf16 operands, fp32 accumulation) for sm_100a.
//
// One persistent thread block per SM walks its range of chunks (gka_common.cuh explains the work
// decomposition).  The block has two "slots"; a slot is a group of 256 threads that owns one chunk of
// C = 64 tokens at a time, so the tensor pipe works on one chunk while the CUDA cores run the
// element-wise part of the other.  Slots take chunks alternately.  An extra warpgroup (kept at 32
// registers by setmaxnreg) holds one issuing thread per slot: every tcgen05.mma of a slot is issued
// there; the slot posts requests to it through an mbarrier and it answers with tcgen05.commit.
//
// Orientation: every product is computed transposed, so that TMEM lanes are channels and TMEM
// columns are tokens (Section 4.2.1 in row form; Algorithm 1 on the whole chunk):
//     S^T[j][c]  = sum_d K[j][d] X'[c][d]                     (M = 64 keys,     N = 64 tokens)
//     P[c][j]    = S^T[j][c] * Gamma[c][j] / zt_c, j <= c      (element-wise, thread = key j)
//     Y^T[d][c]  = sum_e H_0[d][e] X'[c][e] + sum_j K[j][d] P[c][j]   (M = 128 channels, N = 64)
//     x_c <- x_c - (2 w/(L+mu)) (Y_c + lambda_c x_c - q_c) + (w - 1)(x_c - x_c^prev)  (thread = d)
//     O^T[i][c]  = sum_e U_0[i][e] X'[c][e] + sum_j V[j][i] P[c][j]
// with X' = zt_c * x_c in bf16, zt_c = max(zeta_c, 2^-60): the row scaling by zeta_c of the
// inter-chunk term rides on the operand, and the mask factor Gamma[c][j] / zt_c = 2^-G_j (G the
// cumulative log2 gate) is a per-thread constant unless a chunk decays below 2^-60.
//
// State: fp32 masters of H and U live in TMEM (2 x 128 columns) for a whole run; per chunk they are
// read once (bf16 operand copy to shared memory, ||H_0||_F^2), scaled by zeta_C and advanced by
// tensor-core products K^T (w o K) and V^T (w o K).  H runs ahead (it is advanced at the start of a
// chunk), U lags (it is advanced after the chunk's output), so both slots share one pair of masters;
// two mbarrier "tokens" keep the chunks in order.
//
// Operands: K and V tiles arrive by TMA (two 64-column boxes, 128-byte swizzle) and serve both as
// K-major operands (rows = keys) and MN-major operands (rows = channels) without a transposed copy.
#include <cuda.h>
#include <cstdlib>

#include "gka_common.cuh"
#include "gka_tc_util.cuh"

namespace gka {
cudaError_t launch_fwd_tile(const FwdArgs &a, cudaStream_t stream);
namespace {

using namespace tcu;

constexpr int D = 128;
constexpr int C = kChunk;
constexpr int NSLOT = 2;
constexpr int ST = 256;                       // threads per slot
constexpr int kThreadsTc = NSLOT * ST + 128;  // 16 slot warps + one warpgroup that issues the MMAs
constexpr int kRegsSlot = 112, kRegsIssuer = 32;   // register split after setmaxnreg (launch: 96 each)

// ---- shared memory map of one slot (bytes; every operand buffer is 1024-byte aligned)
constexpr uint32_t OFF_K = 0;          // K tile: 2 boxes [64 keys][64 ch], SW128
constexpr uint32_t OFF_V = 16384;      // V tile, same layout
constexpr uint32_t OFF_KW = 32768;     // w o K, same layout
constexpr uint32_t OFF_H = 49152;      // bf16 H_0 (later U_0): 2 halves [128 rows][64 cols], SW128, K-major
constexpr uint32_t OFF_X = 81920;      // X' as B operand: [128 ch (k-rows)][64 tokens], SW128, MN-major
constexpr uint32_t OFF_P = 98304;      // P  as B operand: [64 keys (k-rows)][64 tokens], SW128, MN-major
constexpr uint32_t OFF_SC = 106496;    // per-slot scalars
struct SlotScalars {
    float G2[C];        // cumulative log2 gate
    float lam[C];       // lambda_c (after the adaptive rule, if any)
    float zt[C];        // clamped zeta_c
    float ac[C];        // G2_c - max(G2_c, -60): exponent correction of clamped tokens
    float w[C];         // zeta_C / zeta_j
    float s0[C];        // 2 / (L + mu)
    float omega[C], rho2[C];   // weight schedule state of Algorithm 1
    float dj[C];        // Frobenius increments
    float part[3][2][C];  // partial sums of the Frobenius epilogue: [quantity][column half][key]
    float4 coef[2][C];  // per-iteration (sigma zt, beta, A, -): x' <- A x' - beta x'_prev + sigma zt (q - y)
    float red[8];
    float hh;           // ||H_0||_F^2
    int clamped;        // chunk decays below 2^-60 somewhere
    int req_op;         // request to the MMA issuer
};
constexpr uint32_t SLOT_BYTES = OFF_SC + 7168;
static_assert(sizeof(SlotScalars) <= 7168, "scalar block too large");

// ---- TMEM columns
// H, U: fp32 masters.  Y0 / Y1: the slots' Y^T / O^T accumulators.  Q: the slots' q tiles as packed bf16 pairs
// (32 columns each).  S: the slots' score accumulators, M = 64 rows each, interleaved on lane halves.
constexpr uint32_t TM_H = 0, TM_U = 128, TM_Y0 = 256, TM_Q = 320, TM_Y1 = 384, TM_S = 448;

enum { BAR_TMA = 0, BAR_A, BAR_B, BAR_REQ, BAR_COUNT };   // per-slot mbarriers
enum { OP_FROB = 1, OP_ITER1, OP_ITER1_LAST, OP_ITER2, OP_OUT, OP_EXIT };

#ifdef GKA_TC_TIMING
// Debug build only: event trace of block 0 (thread 0 of each slot and the two issuer threads).
__device__ long long g_trace[4][8192];
__device__ int g_trace_n[4];
__shared__ int s_trace_n[4];
#define TRACE_DECL
#define TRACE(role, id)                                                                                        \
    do {                                                                                                       \
        if (blockIdx.x == 0 && s_trace_n[role] < 8192)                                                         \
            g_trace[role][s_trace_n[role]++] = (clock64() << 8) | (long long)(id);                             \
    } while (0)
#define TSTAMP(k)                   \
    do {                            \
        if (t == 0) TRACE(slot, k); \
    } while (0)
#else
#define TRACE_DECL
#define TRACE(role, id)
#define TSTAMP(k)
#endif

// ---------------------------------------------------------------------------------------------
// MMA issue.  One thread per slot (in the issuer warpgroup) runs the slot's tcgen05.mma batches.  Operand
// descriptors are a base low word per operand plus a compile-time step per k-step (K = 16 per instruction):
//   K-major tiles made of two 64-column boxes: k-step ks -> box ks / 4 (`box` bytes apart), 32 bytes per step;
//   MN-major tiles: 16 k-rows = 2048 bytes per step.
// ---------------------------------------------------------------------------------------------
struct IssueCtx {
    uint32_t base14;              // (shared address of the slot's buffers) >> 4
    uint32_t tm_y, tm_s, bars;
};
// acc = A(K-major, 2 boxes ABOX apart) x B(MN-major) over 8 k-steps; first step overwrites when !ACC0
template <int ACC0, uint32_t A, int ABOX, uint32_t B, int KS = 0>
__device__ __forceinline__ void mma_k8_kmaj_mn(uint32_t d, uint32_t base14, uint32_t idesc) {
    if constexpr (KS < 8) {
        mma_ss<(KS == 0 ? ACC0 : 1), A + kstep(KS, ABOX), B + mnstep(KS)>(d, base14, idesc);
        mma_k8_kmaj_mn<ACC0, A, ABOX, B, KS + 1>(d, base14, idesc);
    }
}
// both operands K-major (8 k-steps); B_OFF is an extra row offset of B in 16-byte units
template <int ACC0, uint32_t A, int ABOX, uint32_t B, int BBOX, uint32_t B_OFF, int KS = 0>
__device__ __forceinline__ void mma_k8_kmaj_kmaj(uint32_t d, uint32_t base14, uint32_t idesc) {
    if constexpr (KS < 8) {
        mma_ss<(KS == 0 ? ACC0 : 1), A + kstep(KS, ABOX), B + kstep(KS, BBOX) + B_OFF>(d, base14, idesc);
        mma_k8_kmaj_kmaj<ACC0, A, ABOX, B, BBOX, B_OFF, KS + 1>(d, base14, idesc);
    }
}
// both operands MN-major over 4 k-steps (64 keys), accumulating
template <uint32_t A, uint32_t B, int KS = 0>
__device__ __forceinline__ void mma_k4_mn_mn(uint32_t d, uint32_t base14, uint32_t idesc) {
    if constexpr (KS < 4) {
        mma_ss<1, A + mnstep(KS), B + mnstep(KS)>(d, base14, idesc);
        mma_k4_mn_mn<A, B, KS + 1>(d, base14, idesc);
    }
}

__device__ __forceinline__ void issuer_run(const IssueCtx &s, int op, uint32_t tm_H, uint32_t tm_U) {
    constexpr uint32_t I_S = make_idesc(64, 64, 0, 1);
    constexpr uint32_t I_Y1 = make_idesc(128, 64, 0, 1);
    constexpr uint32_t I_Y2 = make_idesc(128, 64, 1, 1);
    constexpr uint32_t I_ADV = make_idesc(128, 128, 1, 1);
    constexpr uint32_t I_GR = make_idesc(64, 64, 0, 0);
    constexpr uint32_t K_k = op_kmaj(OFF_K), K_mn = op_mn(OFF_K), V_mn = op_mn(OFF_V), Kw_mn = op_mn(OFF_KW);
    constexpr uint32_t H_k = op_kmaj(OFF_H), X_mn = op_mn(OFF_X), P_mn = op_mn(OFF_P);
    const uint32_t b = s.base14;
    if (op == OP_ITER1 || op == OP_ITER1_LAST) {
        mma_k8_kmaj_mn<0, K_k, 8192, X_mn>(s.tm_s, b, I_S);
        mma_commit(s.bars + 8 * BAR_A);
        if (op == OP_ITER1) mma_k8_kmaj_mn<0, H_k, 16384, X_mn>(s.tm_y, b, I_Y1);
    } else if (op == OP_ITER2) {
        mma_k4_mn_mn<K_mn, P_mn>(s.tm_y, b, I_Y2);
        mma_commit(s.bars + 8 * BAR_B);
    } else if (op == OP_FROB) {
        // H advance: Hm += K^T (w o K)
        mma_k4_mn_mn<K_mn, Kw_mn>(tm_H, b, I_ADV);
        // (K H_0)[:, 0:64] -> Y columns, lanes +0;  (K H_0)[:, 64:128] -> the slot's S region;  Gram -> Y columns, lanes +16
        mma_k8_kmaj_kmaj<0, K_k, 8192, H_k, 16384, 0>(s.tm_y, b, I_GR);
        mma_k8_kmaj_kmaj<0, K_k, 8192, H_k, 16384, (8192u >> 4)>(s.tm_s, b, I_GR);
        mma_k8_kmaj_kmaj<0, K_k, 8192, K_k, 8192, 0>(s.tm_y + (16u << 16), b, I_GR);
        mma_commit(s.bars + 8 * BAR_A);
    } else if (op == OP_OUT) {
        mma_k8_kmaj_mn<0, H_k, 16384, X_mn>(s.tm_y, b, I_Y1);
        mma_k4_mn_mn<V_mn, P_mn>(s.tm_y, b, I_Y2);
        mma_commit(s.bars + 8 * BAR_A);
        mma_k4_mn_mn<V_mn, Kw_mn>(tm_U, b, I_ADV);
        mma_commit(s.bars + 8 * BAR_B);
    }
}

// Everything a slot thread needs to know about itself.
struct SlotCtx {
    int slot, t;                  // slot index, thread in slot (0..255)
    int lane, half, warp_q;       // TMEM lane (0..127), column / token half (0..1), warp % 4
    unsigned char *sptr;          // the slot's shared buffers
    SlotScalars *sc;
    uint32_t bars;                // shared address of the slot's mbarriers
    uint32_t tm_y, tm_s, tm_q;    // accumulator addresses (tm_s includes the slot's lane offset), q tile columns
    uint32_t tm_H, tm_U;          // masters
    uint32_t lane_addr;           // (32 * warp_q) << 16
    uint32_t ph[BAR_COUNT];       // phase parity of each mbarrier
    uint32_t abort_addr;          // shared address of the block's abort flag
};

__device__ __forceinline__ bool slot_aborted(const SlotCtx &cx) {
    int v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(cx.abort_addr) : "memory");
    return v != 0;
}
// Wait for an mbarrier phase: one warp of the slot polls (bounded), the others sleep in the slot's
// named barrier, so waiting warps do not take issue slots from the other slot's working warps.
__device__ __forceinline__ void slot_wait_addr(SlotCtx &cx, uint32_t bar, uint32_t parity) {
    if ((cx.t >> 5) == cx.slot && !slot_aborted(cx)) {   // the polling warp of slot s sits on scheduler s
        if (!mbar_wait_bounded(bar, parity)) {             // the block reports GKA_ERR_TIMEOUT when it ends
            asm volatile("st.shared.b32 [%0], %1;" ::"r"(cx.abort_addr), "r"(1) : "memory");
        }
    }
    slot_sync(cx.slot);
}
__device__ __forceinline__ void slot_wait(SlotCtx &cx, int which) {
    slot_wait_addr(cx, cx.bars + 8 * which, cx.ph[which]);
    cx.ph[which] ^= 1u;
}
// Ask the issuer warp for a batch of MMAs.  Call after slot_sync: every thread's writes and fences are done.
// The issuing thread can stall while the tensor pipe works through earlier batches, which is why it is not
// one of the slot's own threads.
__device__ __forceinline__ void slot_post(SlotCtx &cx, int op) {
    if (cx.t == 0) {
        *reinterpret_cast<volatile int *>(&cx.sc->req_op) = op;
        mbar_arrive(cx.bars + 8 * BAR_REQ);
    }
}

// Masked score epilogue: S^T (TMEM, M = 64 layout, 16 lanes per quadrant) -> P operand in shared memory.
// Every thread of the slot takes part: warp quadrant q covers keys 16 q .. 16 q + 15, column half `half`.
__device__ __forceinline__ void p_epilogue(SlotCtx &cx) {
    const int l = cx.lane & 31;
    const SlotScalars *sc = cx.sc;
    const bool clamped = sc->clamped != 0;
    uint32_t r[16];
    TMEM_LD_16x256b_x4(cx.tm_s + cx.lane_addr + 32 * cx.half, r);
    tmem_wait_ld();
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int j = 16 * cx.warp_q + (l >> 2) + 8 * h;
        const float bj = -sc->G2[j];
        const float invz = ex2_fast(fminf(bj, 126.f));
        unsigned char *prow = cx.sptr + OFF_P + j * 128 + (l & 3) * 4;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c0 = 32 * cx.half + 8 * i + 2 * (l & 3);
            float f0 = invz, f1 = invz;
            if (clamped) {
                f0 = ex2_fast(sc->ac[c0] + bj);
                f1 = ex2_fast(sc->ac[c0 + 1] + bj);
            }
            const float p0 = (j <= c0) ? __uint_as_float(r[4 * i + 2 * h]) * f0 : 0.f;
            const float p1 = (j <= c0 + 1) ? __uint_as_float(r[4 * i + 2 * h + 1]) * f1 : 0.f;
            const int chunk = (4 * cx.half + i) ^ (j & 7);
            *reinterpret_cast<uint32_t *>(prow + chunk * 16) = pack_bf16(p0, p1);
        }
    }
}

// One pass over a master (H or U) for this thread's row and column half: source is TMEM, or global memory
// at the start of a run.  Writes the bf16 operand copy, optionally accumulates the sum of squares, scales
// by zeta_C and stores the result back to TMEM.
template <bool SUMSQ>
__device__ __forceinline__ float master_pass(SlotCtx &cx, uint32_t tm_master, bool from_global, const float *grow,
                                             float zetaC) {
    float ss = 0.f;
    unsigned char *hrow = cx.sptr + OFF_H + cx.half * 16384 + cx.lane * 128;
#pragma unroll
    for (int piece = 0; piece < 2; ++piece) {
        uint32_t r[32];
        const uint32_t taddr = tm_master + cx.lane_addr + 64 * cx.half + 32 * piece;
        if (!from_global) {
            TMEM_LD32(taddr, r);
            tmem_wait_ld();
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float4 v4 = grow ? ldg_stream_f32x4(grow + 64 * cx.half + 32 * piece + 4 * i)
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
                r[4 * i + 0] = __float_as_uint(v4.x); r[4 * i + 1] = __float_as_uint(v4.y);
                r[4 * i + 2] = __float_as_uint(v4.z); r[4 * i + 3] = __float_as_uint(v4.w);
            }
        }
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
            uint32_t pk[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float v0 = __uint_as_float(r[8 * ch + 2 * u]), v1 = __uint_as_float(r[8 * ch + 2 * u + 1]);
                if (SUMSQ) ss = fmaf(v0, v0, fmaf(v1, v1, ss));
                pk[u] = pack_bf16(v0, v1);
            }
            const int chunk = (4 * piece + ch) ^ (cx.lane & 7);
            *reinterpret_cast<uint4 *>(hrow + chunk * 16) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * zetaC);
        TMEM_ST32(taddr, r);
    }
    tmem_wait_st();
    return ss;
}

// Copy this thread's part of a master from TMEM to global memory (final state of a sequence).
__device__ __forceinline__ void master_store(SlotCtx &cx, uint32_t tm_master, float *grow) {
#pragma unroll
    for (int piece = 0; piece < 2; ++piece) {
        uint32_t r[32];
        TMEM_LD32(tm_master + cx.lane_addr + 64 * cx.half + 32 * piece, r);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 8; ++i)
            *reinterpret_cast<float4 *>(grow + 64 * cx.half + 32 * piece + 4 * i) =
                make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]), __uint_as_float(r[4 * i + 2]),
                            __uint_as_float(r[4 * i + 3]));
    }
}

// The solve of one chunk: x_0, n_iter Chebyshev iterations, and the masked scores of the final iterate.
// Kept out of line on purpose: the iterate (x, x_prev: 64 registers per thread) must stay in registers for
// the whole loop, and a call boundary makes the compiler park the caller's chunk-level values once per
// chunk instead of reloading spilled values inside the loop (local memory misses the small L1 here).
// Returns the updated phase parities of the slot's barriers A and B (bit 0, bit 1).
__device__ __forceinline__ uint32_t chunk_solve(SlotCtx cx, int n_iter) {
    SlotScalars *sc = cx.sc;
    const int slot = cx.slot, t = cx.t, lane = cx.lane, half = cx.half;
    TRACE_DECL;
    // ---- x_0 = 2 q / (L + mu), X' operand (this thread: channel `lane`, tokens 32 half .. 32 half + 31)
    float xm[32];
    uint32_t dl[16];      // x_i - x_{i-1} as packed bf16 pairs: the momentum term shrinks as the iteration converges
    {
        uint32_t qp[16];
        TMEM_LD16(cx.tm_q + cx.lane_addr + 16 * half, qp);
        tmem_wait_ld();
        unsigned char *xrow = cx.sptr + OFF_X + lane * 128;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
            uint32_t pk[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i0 = 8 * ch + 2 * u, c0 = 32 * half + i0;
                // the iterate is kept scaled by zt_c (the recurrence is linear), as the operand needs it
                const float x0 = sc->s0[c0] * sc->zt[c0] * bf16_lo(qp[i0 >> 1]);
                const float x1 = sc->s0[c0 + 1] * sc->zt[c0 + 1] * bf16_hi(qp[i0 >> 1]);
                xm[i0] = x0; xm[i0 + 1] = x1;
                dl[i0 >> 1] = pack_bf16(x0, x1);     // x_{-1} = 0 (Algorithm 1), so the first difference is x_0
                pk[u] = dl[i0 >> 1];
            }
            *reinterpret_cast<uint4 *>(xrow + (((4 * half + ch) ^ (lane & 7)) * 16)) =
                make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
    }
    fence_async_smem();
    fence_before();
    slot_sync(slot);
    TSTAMP(6);

    // ---- Algorithm 1: n_iter iterations on the whole chunk (+ one extra score pass for the output)
    for (int it = 0; it <= n_iter; ++it) {
        const bool last = (it == n_iter);
        slot_post(cx, last ? OP_ITER1_LAST : OP_ITER1);
        TSTAMP(17);
        if (!last && t < C) {   // weight schedule and per-token coefficients of this iteration
            const float omega = 4.f / (4.f - sc->rho2[t] * sc->omega[t]);
            sc->omega[t] = omega;
            const float sigma = sc->s0[t] * omega, beta = omega - 1.f;
            sc->coef[it & 1][t] = make_float4(sigma * sc->zt[t], beta, sigma * sc->lam[t], 0.f);
        }
        TSTAMP(15);
        slot_wait(cx, BAR_A);
        fence_after();
        TSTAMP(7);
        p_epilogue(cx);
        fence_async_smem();
        fence_before();
        slot_sync(slot);
        TSTAMP(8);
        if (last) break;
        slot_post(cx, OP_ITER2);
        TSTAMP(16);
        slot_wait(cx, BAR_B);
        fence_after();
        TSTAMP(9);
        {
            const float4 *coef = sc->coef[it & 1] + 32 * half;
            unsigned char *xrow = cx.sptr + OFF_X + lane * 128;
#pragma unroll
            for (int piece = 0; piece < 8; ++piece) {     // 4 tokens at a time keeps the transient registers few
                uint32_t r[4], qq[2];
                TMEM_LD4(cx.tm_y + cx.lane_addr + 32 * half + 4 * piece, r);
                TMEM_LD2(cx.tm_q + cx.lane_addr + 16 * half + 2 * piece, qq);
                tmem_wait_ld();
                uint32_t pk[2];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    float dn[2];
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int i = 4 * piece + 2 * u + e;
                        const float4 cf = coef[i];
                        const float qv = e == 0 ? bf16_lo(qq[u]) : bf16_hi(qq[u]);
                        const float dv = e == 0 ? bf16_lo(dl[i >> 1]) : bf16_hi(dl[i >> 1]);
                        const float acc = __uint_as_float(r[2 * u + e]);
                        // x_{i+1} - x_i = beta (x_i - x_{i-1}) + sigma (q - A x_i), with the lambda part of A explicit
                        dn[e] = fmaf(cf.x, qv - acc, fmaf(cf.y, dv, -cf.z * xm[i]));
                        xm[i] += dn[e];
                    }
                    dl[(4 * piece + 2 * u) >> 1] = pack_bf16(dn[0], dn[1]);
                    pk[u] = pack_bf16(xm[4 * piece + 2 * u], xm[4 * piece + 2 * u + 1]);
                }
                const int chunk = (4 * half + (piece >> 1)) ^ (lane & 7);
                *reinterpret_cast<uint2 *>(xrow + chunk * 16 + 8 * (piece & 1)) = make_uint2(pk[0], pk[1]);
            }
        }
        fence_async_smem();
        fence_before();
        slot_sync(slot);
        TSTAMP(10);
    }

    return cx.ph[BAR_A] | (cx.ph[BAR_B] << 1);
}

__global__ void __launch_bounds__(kThreadsTc, 1)
fwd_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, FwdArgs a) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_bars[NSLOT * BAR_COUNT + 2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    unsigned char *smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    const int tid = threadIdx.x;

    if (tid == 0) {
        s_abort = 0;
#ifdef GKA_TC_TIMING
        for (int i = 0; i < 4; ++i) s_trace_n[i] = 0;
#endif
        for (int i = 0; i < NSLOT * BAR_COUNT + 2; ++i)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s_bars[i])));
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
    const uint32_t tm_H = tmem + TM_H, tm_U = tmem + TM_U;
    const uint32_t tokH = smem_u32(&s_bars[NSLOT * BAR_COUNT]);
    const uint32_t tokU = tokH + 8;
    TRACE_DECL;

    const WorkPlan &P = a.plan;
    const int item = blockIdx.x;
    const long long f_lo = P.lo(item), f_hi = P.lo(item + 1);
    const int n_mine = (int)(f_hi - f_lo);          // chunks of this block

    if (tid >= NSLOT * ST) {
        // ================================ MMA issuer warpgroup ================================
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsIssuer));
        const int s = ((tid - NSLOT * ST) >> 5) - 2;    // warps 2, 3 of the warpgroup (schedulers 2, 3) serve slots 0, 1
        if ((tid & 31) == 0 && s >= 0 && f_lo + s < f_hi) {
            const SlotScalars *isc = reinterpret_cast<const SlotScalars *>(smem + (size_t)s * SLOT_BYTES + OFF_SC);
            const uint32_t sb = smem_u32(smem + (size_t)s * SLOT_BYTES);
            IssueCtx ic;
            ic.base14 = (sb >> 4) & 0x3FFF;   // K, H_0 / U_0 are used K-major; K, V, w o K, X', P MN-major (8192 bytes
                                              // from one group of 64 channels or tokens to the next)
            ic.tm_y = tmem + (s == 0 ? TM_Y0 : TM_Y1);
            ic.tm_s = tmem + TM_S + ((uint32_t)(16 * s) << 16);
            ic.bars = smem_u32(&s_bars[s * BAR_COUNT]);
            uint32_t reqph = 0;
            for (;;) {
                // a request normally arrives within microseconds; give up after seconds of silence
                bool got = false;
                for (int tries = 0; tries < 4 && !got; ++tries) got = mbar_spin_bounded(ic.bars + 8 * BAR_REQ, reqph);
                if (!got || s_abort != 0) {
                    s_abort = 1;
                    break;
                }
                reqph ^= 1u;
                const int op = *reinterpret_cast<const volatile int *>(&isc->req_op);
                TRACE(2 + s, 32 + op);
                if (op == OP_EXIT) break;
                fence_after();
                issuer_run(ic, op, tm_H, tm_U);
                TRACE(2 + s, 48 + op);
            }
        }
    } else {
        // ================================= slot threads =================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSlot));
        SlotCtx cx;
        cx.slot = tid / ST;
        cx.t = tid % ST;
        cx.lane = cx.t & 127;
        cx.half = cx.t >> 7;
        cx.warp_q = (cx.t >> 5) & 3;
        cx.sptr = smem + (size_t)cx.slot * SLOT_BYTES;
        cx.sc = reinterpret_cast<SlotScalars *>(cx.sptr + OFF_SC);
        cx.bars = smem_u32(&s_bars[cx.slot * BAR_COUNT]);
        cx.lane_addr = (uint32_t)(32 * cx.warp_q) << 16;
#pragma unroll
        for (int i = 0; i < BAR_COUNT; ++i) cx.ph[i] = 0;
        cx.abort_addr = smem_u32(&s_abort);
        cx.tm_y = tmem + (cx.slot == 0 ? TM_Y0 : TM_Y1);
        cx.tm_q = tmem + TM_Q + 32 * cx.slot;
        cx.tm_s = tmem + TM_S + ((uint32_t)(16 * cx.slot) << 16);
        cx.tm_H = tm_H;
        cx.tm_U = tm_U;
        SlotScalars *sc = cx.sc;
        const int slot = cx.slot, t = cx.t, lane = cx.lane, half = cx.half;
        const uint32_t sbase = smem_u32(cx.sptr);

        const __nv_bfloat16 *gq = reinterpret_cast<const __nv_bfloat16 *>(a.q);
        __nv_bfloat16 *gout = reinterpret_cast<__nv_bfloat16 *>(a.out);
        const size_t st = state_floats(D, D);
        const bool adaptive = (a.flags & GKA_FLAG_ADAPTIVE_LAMBDA) != 0;

        auto issue_tma = [&](long long f) {   // thread 0 of the slot: K and V tiles of flat chunk f
            const int seq = (int)(f / P.N), n = (int)(f % P.N);
            const int b = seq / a.heads, h = seq % a.heads;
            const int y = b * a.T + n * C;
            const uint32_t bar = cx.bars + 8 * BAR_TMA;
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(32768u) : "memory");
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int x = h * D + 64 * hf;
                asm volatile(
                    "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::
                        "r"(sbase + OFF_K + 8192 * hf), "l"(reinterpret_cast<uint64_t>(&tmK)), "r"(x), "r"(y), "r"(bar)
                    : "memory");
                asm volatile(
                    "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::
                        "r"(sbase + OFF_V + 8192 * hf), "l"(reinterpret_cast<uint64_t>(&tmV)), "r"(x), "r"(y), "r"(bar)
                    : "memory");
            }
        };

        if (t == 0 && f_lo + slot < f_hi) issue_tma(f_lo + slot);
        slot_sync(slot);

        for (int m = slot; m < n_mine; m += NSLOT) {       // m: index of this chunk inside the block's range
            const long long f = f_lo + m;
            const int seq = (int)(f / P.N), n = (int)(f % P.N);
            const int b = seq / a.heads, h = seq % a.heads;
            const size_t tok0 = ((size_t)b * a.T + (size_t)n * C) * a.heads + h;
            const bool run_start = (m == 0) || (n == 0);
            const bool seq_end = (n == P.N - 1);
            const float *init_src = nullptr;           // where a run's start state comes from (nullptr = zero)
            if (run_start) init_src = (n == 0) ? (a.state_in ? a.state_in + (size_t)seq * st : nullptr)
                                               : a.ws.start + (size_t)item * st;

            // ---- q for this thread's channel and its 32 tokens, packed bf16 pairs (issued early)
            {
                uint32_t qp[16];
                const unsigned short *qs = reinterpret_cast<const unsigned short *>(gq) +
                                           (tok0 + (size_t)32 * half * a.heads) * D + lane;
                const size_t rs = (size_t)a.heads * D;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const uint32_t lo = ldg_stream_u16(qs + (size_t)(2 * i) * rs), hi = ldg_stream_u16(qs + (size_t)(2 * i + 1) * rs);
                    qp[i] = lo | (hi << 16);
                }
                // parked in TMEM for the whole chunk (exact: q is bf16); this slot's previous chunk is done with it
                TMEM_ST16(cx.tm_q + cx.lane_addr + 16 * half, qp);
                tmem_wait_st();
            }

            // ---- gates (threads 0..63 own token c = t for scalar bookkeeping)
            if (t < C) {
                const float g = ldg_stream_f32(a.gate + tok0 + (size_t)t * a.heads);
                sc->w[t] = fmaxf(log2f(g), -115.f);     // temporary: log2 gamma
                sc->lam[t] = ldg_stream_f32(a.lam + tok0 + (size_t)t * a.heads);
            }
            slot_sync(slot);
            float G2c = 0.f;
            if (t < C) {
                for (int i = 0; i <= t; ++i) G2c += sc->w[i];
            }
            slot_sync(slot);
            if (t < C) {
                sc->G2[t] = G2c;
                const float mc = fmaxf(G2c, -60.f);
                sc->zt[t] = exp2f(mc);
                sc->ac[t] = G2c - mc;
                if (t == C - 1) sc->clamped = (G2c < -60.f) ? 1 : 0;
            }
            slot_sync(slot);
            if (t < C) sc->w[t] = exp2f(sc->G2[C - 1] - sc->G2[t]);
            const float zetaC = exp2f(sc->G2[C - 1]);
            slot_sync(slot);
            TSTAMP(0);

            // ---- K, V tiles have landed
            slot_wait(cx, BAR_TMA);
            TSTAMP(1);

            // ---- w o K (same swizzled positions as K)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int qi = t + ST * i;                 // 16-byte chunk index in the 16 KB tile
                const int j = (qi & 511) >> 3;             // key row of this chunk
                uint4 v = *reinterpret_cast<const uint4 *>(cx.sptr + OFF_K + qi * 16);
                const float wj = sc->w[j];
                uint32_t *pv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
                for (int u = 0; u < 4; ++u) pv[u] = pack_bf16(bf16_lo(pv[u]) * wj, bf16_hi(pv[u]) * wj);
                *reinterpret_cast<uint4 *>(cx.sptr + OFF_KW + qi * 16) = v;
            }
            TSTAMP(2);

            // ---- H master: wait for the previous chunk's advance, then one pass: ||H_0||^2, bf16 copy, scale
            if (m > 0) slot_wait_addr(cx, tokH, (uint32_t)((m - 1) & 1));   // chunk m - 1 finished its H work
            fence_after();
            {
                float hh = master_pass<true>(cx, tm_H, run_start,
                                             init_src ? init_src + (size_t)lane * D : nullptr, zetaC);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) hh += __shfl_xor_sync(0xffffffffu, hh, o);
                if ((t & 31) == 0) sc->red[t >> 5] = hh;
            }
            fence_async_smem();
            fence_before();
            slot_sync(slot);
            slot_post(cx, OP_FROB);
            if (t == 0) {
                float s = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) s += sc->red[i];
                sc->hh = s;
            }
            TSTAMP(3);
            slot_wait(cx, BAR_A);
            fence_after();
            TSTAMP(4);

            // ---- chunk-wise Frobenius norms: partial sums per key from K H_0 and the Gram matrix.
            // 32x32b loads address whole 32-lane quadrants; an M = 64 accumulator placed at lane offset 0 / 16
            // has its rows on lanes 0..15 / 16..31 of every quadrant.  Each thread takes 32 of the 64 columns.
            {
                const int l = lane & 31;
                const int j = 16 * cx.warp_q + (l & 15);
                const uint32_t y_cols = cx.tm_y + cx.lane_addr + 32 * half;
                const uint32_t s_cols = tmem + TM_S + cx.lane_addr + 32 * half;
                float a0 = 0.f, a1 = 0.f, bjs = 0.f;
#pragma unroll
                for (int src = 0; src < 2; ++src) {     // (K H_0) columns 0..63 (Y region) and 64..127 (S region)
                    uint32_t r[32];
                    TMEM_LD32(src == 0 ? y_cols : s_cols, r);
                    tmem_wait_ld();
                    const unsigned char *krow = cx.sptr + OFF_K + src * 8192 + j * 128;
                    float acc = 0.f;
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        const int chunk = (4 * half + ch) ^ (j & 7);
                        const uint4 kv = *reinterpret_cast<const uint4 *>(krow + chunk * 16);
                        const uint32_t *pk = reinterpret_cast<const uint32_t *>(&kv);
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            acc = fmaf(__uint_as_float(r[8 * ch + 2 * u]), bf16_lo(pk[u]), acc);
                            acc = fmaf(__uint_as_float(r[8 * ch + 2 * u + 1]), bf16_hi(pk[u]), acc);
                        }
                    }
                    if (src == 0) a0 = acc; else a1 = acc;
                }
                const float G2j = sc->G2[j];
                {
                    uint32_t r[32];
                    TMEM_LD32(y_cols, r);                // Gram rows sit on lanes 16..31 of the Y columns
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int ii = 32 * half + i;
                        const float g = __uint_as_float(r[i]);
                        const float g2 = g * g;
                        if (ii < j) bjs = fmaf(2.f * ex2_fast(G2j - sc->G2[ii]), g2, bjs);
                        else if (ii == j) bjs += g2;
                    }
                }
                if ((l >> 4) == 0) sc->part[0][half][j] = a0;
                if ((l >> 4) == slot) sc->part[1][half][j] = a1;
                if ((l >> 4) == 1) sc->part[2][half][j] = bjs;
            }
            fence_before();
            slot_sync(slot);
            // H master is final for this chunk, the Frobenius temporaries are consumed
            if (seq_end && a.state_out) {
                fence_after();
                master_store(cx, tm_H, a.state_out + (size_t)seq * st + (size_t)lane * D);
                fence_before();
                slot_sync(slot);
            }
            if (t == 0) mbar_arrive(tokH);
            TSTAMP(5);

            // ---- f_c, Chebyshev initialisation (threads 0..63: token c = t)
            if (t < C) {
                sc->dj[t] = fmaf(2.f * exp2f(sc->G2[t]),
                                 (sc->part[0][0][t] + sc->part[0][1][t]) + (sc->part[1][0][t] + sc->part[1][1][t]),
                                 sc->part[2][0][t] + sc->part[2][1][t]);
            }
            slot_sync(slot);
            if (t < C) {
                const float G2t = sc->G2[t];
                float s = exp2f(2.f * G2t) * sc->hh;
                for (int j = 0; j <= t; ++j) s = fmaf(ex2_fast(2.f * (G2t - sc->G2[j])), sc->dj[j], s);
                const float fc = sqrtf(fmaxf(s, 0.f));
                float lamc = sc->lam[t];
                if (adaptive) lamc *= fc;
                const float Lpm = fc + 2.f * lamc;
                const float rho = fc / Lpm;
                sc->lam[t] = lamc;
                sc->rho2[t] = rho * rho;
                sc->omega[t] = 2.f;
                sc->s0[t] = 2.f / Lpm;
                if (a.fro_out) a.fro_out[tok0 + (size_t)t * a.heads] = fc;
            }
            slot_sync(slot);

            // ---- x_0, Chebyshev iterations, final masked scores
            {
                const uint32_t phab = chunk_solve(cx, a.n_iter);
                cx.ph[BAR_A] = phab & 1u;
                cx.ph[BAR_B] = phab >> 1;
            }

            // ---- output: U master pass (bf16 copy into the H buffer, scale), O^T = U_0 X'^T + V^T P^T, U advance
            if (m > 0) slot_wait_addr(cx, tokU, (uint32_t)((m - 1) & 1));   // chunk m - 1 wrote its output, advanced U
            fence_after();
            master_pass<false>(cx, tm_U, run_start,
                               init_src ? init_src + (size_t)D * D + (size_t)lane * D : nullptr, zetaC);
            fence_async_smem();
            fence_before();
            slot_sync(slot);
            slot_post(cx, OP_OUT);
            TSTAMP(11);
            slot_wait(cx, BAR_A);
            fence_after();
            TSTAMP(12);
            {
                unsigned short *orow = reinterpret_cast<unsigned short *>(gout) +
                                       (tok0 + (size_t)32 * half * a.heads) * D + lane;
                const size_t rs = (size_t)a.heads * D;
#pragma unroll
                for (int piece = 0; piece < 2; ++piece) {
                    uint32_t r[16];
                    TMEM_LD16(cx.tm_y + cx.lane_addr + 32 * half + 16 * piece, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const __nv_bfloat16 ob = __float2bfloat16_rn(__uint_as_float(r[i]));
                        orow[(size_t)(16 * piece + i) * rs] = *reinterpret_cast<const unsigned short *>(&ob);
                    }
                }
            }
            TSTAMP(13);
            slot_wait(cx, BAR_B);     // U advance done: every tensor-core read of this chunk's tiles is done
            fence_after();
            if (seq_end && a.state_out)
                master_store(cx, tm_U, a.state_out + (size_t)seq * st + (size_t)D * D + (size_t)lane * D);
            fence_before();
            slot_sync(slot);
            if (t == 0) {
                mbar_arrive(tokU);
                if (f + NSLOT < f_hi && !slot_aborted(cx)) issue_tma(f + NSLOT);
            }
            TSTAMP(14);
            if (slot_aborted(cx)) break;
        }
        if (f_lo + slot < f_hi) slot_post(cx, OP_EXIT);
    }

#ifdef GKA_TC_TIMING
    __syncthreads();
    if (blockIdx.x == 0 && tid < 4) g_trace_n[tid] = s_trace_n[tid];
#endif
    fence_before();
    __syncthreads();
    if (tid == 0 && s_abort != 0 && a.device_status) atomicExch(a.device_status, (int)GKA_ERR_TIMEOUT);
    if (tid < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
}

// ---------------------------------------------------------------------------------------------
// Segment summaries on the tensor cores: for every work item whose range ends inside a sequence, the decay
// product and (delta-H, delta-U) of its last run, i.e. the run's final state for a zero start state:
//     dH = sum_j w_j k_j k_j^T,   dU = sum_j w_j v_j k_j^T,   w_j = prod of the gates after token j in the run.
// The weights are formed in log2 space from the run's total log-decay (one pre-pass over the gates) and a
// running prefix, so every chunk is a pure accumulation K^T (w o K), V^T (w o K) into TMEM: no rescaling pass
// and no wait between chunks.  One block of 128 threads per item; K/V tiles in 4 stages, w o K in 2.
// ---------------------------------------------------------------------------------------------
constexpr int SUM_NS = 4;
constexpr uint32_t SUM_STAGE = 32768;                   // K tile + V tile
constexpr uint32_t SUM_OFF_KW = SUM_NS * SUM_STAGE;     // 2 x (w o K)
constexpr uint32_t SUM_SMEM = SUM_OFF_KW + 2 * 16384 + 1024;

__global__ void __launch_bounds__(128, 1)
fwd_tc_summary_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, FwdArgs a) {
    const WorkPlan &P = a.plan;
    const int item = blockIdx.x;
    if (!P.cut_out(item)) return;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_bars[SUM_NS + 2];      // TMA stages, MMA parity 0 / 1
    __shared__ uint32_t s_tmem_base;
    __shared__ float s_w[C], s_red[4];
    unsigned char *smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    const uint32_t sb = smem_u32(smem);
    const int t = threadIdx.x, warp_q = t >> 5, l = t & 31;
    const uint32_t lane_addr = (uint32_t)(32 * warp_q) << 16;

    if (t == 0) {
        for (int i = 0; i < SUM_NS + 2; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s_bars[i])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (t < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(smem_u32(&s_tmem_base))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = s_tmem_base, tm_H = tmem, tm_U = tmem + 128;

    const long long f0 = P.last_run_start(item), f1 = P.lo(item + 1);
    const int nch = (int)(f1 - f0);
    const int seq = (int)(f0 / P.N), b = seq / a.heads, h = seq % a.heads;
    const int n0 = (int)(f0 % P.N);                        // first chunk of the run inside its sequence
    const float *grun = a.gate + ((size_t)b * a.T + (size_t)n0 * C) * a.heads + h;   // token stride: heads
    auto issue_tma = [&](int n) {
        const int stage = n % SUM_NS;
        const int y = b * a.T + (n0 + n) * C;
        const uint32_t bar = smem_u32(&s_bars[stage]);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(32768u) : "memory");
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            const int x = h * D + 64 * hf;
            asm volatile(
                "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::
                    "r"(sb + stage * SUM_STAGE + 8192 * hf), "l"(reinterpret_cast<uint64_t>(&tmK)), "r"(x), "r"(y), "r"(bar)
                : "memory");
            asm volatile(
                "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::
                    "r"(sb + stage * SUM_STAGE + 16384 + 8192 * hf), "l"(reinterpret_cast<uint64_t>(&tmV)), "r"(x), "r"(y),
                "r"(bar)
                : "memory");
        }
    };
    if (t == 0)
        for (int n = 0; n < nch && n < SUM_NS; ++n) issue_tma(n);

    // ---- pre-pass: total log2 decay of the run
    float total = 0.f;
    {
        float s = 0.f;
        for (int i = t; i < nch * C; i += 128) s += fmaxf(log2f(grun[(size_t)i * a.heads]), -115.f);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (l == 0) s_red[warp_q] = s;
        __syncthreads();
        total = s_red[0] + s_red[1] + s_red[2] + s_red[3];
        __syncthreads();
    }

    auto load_lg = [&](int n) -> float {   // threads 0..63: log2 gate of token t of chunk n
        return (t < C && n < nch) ? fmaxf(log2f(grun[((size_t)n * C + t) * a.heads]), -115.f) : 0.f;
    };
    float lg_cur = load_lg(0);
    float prefix = 0.f;                    // log2 decay of the chunks before the current one
    bool failed = false;
    constexpr uint32_t I_ADV = make_idesc(128, 128, 1, 1);
    for (int n = 0; n < nch && !failed; ++n) {
        const int stage = n % SUM_NS, par = n & 1;
        const float lg_next = load_lg(n + 1);
        if (n >= 2) {   // the MMAs of chunk n - 2 are done: its w o K buffer and its tile stage are free
            if (!mbar_wait_bounded(smem_u32(&s_bars[SUM_NS + par]), (uint32_t)(((n - 2) >> 1) & 1))) failed = true;
            if (t == 0 && n + 2 < nch) issue_tma(n + 2);
        }
        // inclusive prefix of the chunk's log2 gates over 64 tokens (two warps), chunk total
        float incl = lg_cur;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float up = __shfl_up_sync(0xffffffffu, incl, o);
            if (l >= o) incl += up;
        }
        if (t == 31) s_red[0] = incl;
        __syncthreads();
        if (t >= 32 && t < C) incl += s_red[0];
        if (t == C - 1) s_red[1] = incl;
        __syncthreads();
        const float chunk_total = s_red[1];
        // w_j = 2^(decay from token j to the end of the run) = 2^((total - prefix) - incl_j)
        if (t < C) s_w[t] = exp2f((total - prefix) - incl);
        prefix += chunk_total;
        __syncthreads();
        if (!mbar_wait_bounded(smem_u32(&s_bars[stage]), (uint32_t)((n / SUM_NS) & 1))) failed = true;
        const unsigned char *kt = smem + stage * SUM_STAGE;
        unsigned char *kw = smem + SUM_OFF_KW + par * 16384;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int qi = t + 128 * i;
            const int j = (qi & 511) >> 3;
            uint4 v = *reinterpret_cast<const uint4 *>(kt + qi * 16);
            const float wj = s_w[j];
            uint32_t *pv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
            for (int u = 0; u < 4; ++u) pv[u] = pack_bf16(bf16_lo(pv[u]) * wj, bf16_hi(pv[u]) * wj);
            *reinterpret_cast<uint4 *>(kw + qi * 16) = v;
        }
        fence_async_smem();
        __syncthreads();
        if (t == 0) {
            fence_after();
            const uint32_t k_mn = desc_lo(sb + stage * SUM_STAGE, 8192), v_mn = desc_lo(sb + stage * SUM_STAGE + 16384, 8192);
            const uint32_t kw_mn = desc_lo(sb + SUM_OFF_KW + par * 16384, 8192);
            if (n == 0) {
                mma_ss_r<0>(tm_H, k_mn, mnstep(0), kw_mn, mnstep(0), I_ADV);
                mma_ss_r<0>(tm_U, v_mn, mnstep(0), kw_mn, mnstep(0), I_ADV);
            } else {
                mma_ss_r<1>(tm_H, k_mn, mnstep(0), kw_mn, mnstep(0), I_ADV);
                mma_ss_r<1>(tm_U, v_mn, mnstep(0), kw_mn, mnstep(0), I_ADV);
            }
#pragma unroll
            for (int ks = 1; ks < 4; ++ks) {
                mma_ss_r<1>(tm_H, k_mn, mnstep(ks), kw_mn, mnstep(ks), I_ADV);
                mma_ss_r<1>(tm_U, v_mn, mnstep(ks), kw_mn, mnstep(ks), I_ADV);
            }
            mma_commit(smem_u32(&s_bars[SUM_NS + par]));
        }
        lg_cur = lg_next;
    }
    // the last two chunks' MMAs
    for (int n = (nch >= 2 ? nch - 2 : 0); n < nch && !failed; ++n)
        if (!mbar_wait_bounded(smem_u32(&s_bars[SUM_NS + (n & 1)]), (uint32_t)((n >> 1) & 1))) failed = true;
    fence_after();
    if (failed) {
        if (t == 0 && a.device_status) atomicExch(a.device_status, (int)GKA_ERR_TIMEOUT);
    } else {
        const size_t st = state_floats(D, D);
        float *dst = a.ws.delta + (size_t)item * st + (size_t)t * D;     // row t of dH, then row t of dU
#pragma unroll
        for (int piece = 0; piece < 8; ++piece) {
            uint32_t r[32];
            TMEM_LD32(tmem + lane_addr + 32 * piece, r);
            tmem_wait_ld();
            float *p = dst + (piece >> 2) * (size_t)D * D + 32 * (piece & 3);
#pragma unroll
            for (int i = 0; i < 8; ++i)
                *reinterpret_cast<float4 *>(p + 4 * i) = make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]),
                                                                     __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
        }
        if (t == 0) a.ws.decay[item] = exp2f(total);
    }
    fence_before();
    __syncthreads();
    if (t < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
}

}  // namespace

bool fwd_tc_available() { return get_encode_fn() != nullptr; }

cudaError_t launch_fwd_tc(const FwdArgs &a, cudaStream_t stream) {
    alignas(64) CUtensorMap tmK, tmV;
    const int rows = a.B * a.T, cols = a.heads * D;
    if (!make_tile_map(&tmK, a.k, rows, cols, 64) || !make_tile_map(&tmV, a.v, rows, cols, 64))
        return cudaErrorInvalidValue;
    cudaError_t err = cudaSuccess;
    bool any_cut = false;
    for (int i = 0; i + 1 < a.plan.G; ++i) any_cut |= a.plan.cut_out(i);
    if (any_cut) {
        err = cudaFuncSetAttribute(fwd_tc_summary_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SUM_SMEM);
        if (err != cudaSuccess) return err;
        fwd_tc_summary_kernel<<<a.plan.G, 128, SUM_SMEM, stream>>>(tmK, tmV, a);
        err = launch_fwd_scan(a, (int)state_floats(D, D), stream);
        if (err != cudaSuccess) return err;
    }
    if (!getenv("GKA_TC_OLD")) return launch_fwd_tile(a, stream);
    const size_t smem = (size_t)NSLOT * SLOT_BYTES + 1024;
    err = cudaFuncSetAttribute(fwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    if (a.ev_start) cudaEventRecord(a.ev_start, stream);
    fwd_tc_kernel<<<a.plan.G, kThreadsTc, smem, stream>>>(tmK, tmV, a);
    if (a.ev_stop) cudaEventRecord(a.ev_stop, stream);
    return cudaGetLastError();
}

#ifdef GKA_TC_TIMING
extern "C" int gka_debug_tc_trace(long long *out /* 4 x 8192 */, int *counts /* 4 */) {
    if (cudaMemcpyFromSymbol(out, g_trace, sizeof(long long) * 4 * 8192) != cudaSuccess) return 1;
    if (cudaMemcpyFromSymbol(counts, g_trace_n, sizeof(int) * 4) != cudaSuccess) return 1;
    return 0;
}
#endif

}  // namespace gka
