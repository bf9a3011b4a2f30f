// tcgen05 / TMEM solve kernel of the chunk-wise GKA forward (bf16 operands, fp32 accumulation) for sm_100a.
//
// Input: for every tile of 128 consecutive tokens of a sequence, the bf16 copies of the tile-initial states
// H_0, U_0 and ||H_0||_F^2 (written by the state kernel, gka_tc_state.cu).  Tiles are independent problems.  Two
// persistent thread blocks share an SM, each with one tile in flight (half of the SM's shared memory and tensor
// memory each), so that the tensor-core products of one block run under the CUDA-core epilogues of the other
// without any coupling in the code.  A tile puts one token on each TMEM lane; every product of the chunk-wise
// form (Section 4.2.1; Algorithm 1 on the whole tile) is an M = 128 tile.
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
// Warp roles: 8 compute warps (warp quadrant q = TMEM lanes 32 q .. 32 q + 31, column half hf = 64 of the 128
// columns: a thread holds one token's 64 channels of the iterate in registers); one warp prepares the gate scalars
// one tile ahead; one thread issues the TMA loads and stores of the tiles; one thread issues every tcgen05.mma.
// The compute warps hand work over through mbarriers (one arrival per warp) and wait for tcgen05.commit.
#include <cuda.h>

#include "gka_common.cuh"
#include "gka_tc_mma.cuh"

namespace gka {
namespace {

using namespace tcu;

constexpr int D = 128;
constexpr int NT = kTile;                  // tokens per tile: one per TMEM lane
constexpr int CT = 256;                    // compute threads
constexpr int NW = CT / 32;                // compute warps
constexpr int kThreadsSolve = CT + 128;    // + helper warpgroup: gate scalars, TMA, MMA issue
constexpr int kBlocksPerSM = 2;
constexpr int kRegsLaunch = 80, kRegsCompute = 104, kRegsHelper = 32;   // register split after setmaxnreg
static_assert(kThreadsSolve * kRegsLaunch * kBlocksPerSM <= 65536, "launch registers");
static_assert(CT * kRegsCompute + 128 * kRegsHelper <= kThreadsSolve * kRegsLaunch, "register split exceeds the launch allocation");

// ---- shared memory map (bytes; operand buffers 1024-byte aligned): three operand tiles and the scalars
constexpr uint32_t BUF_K = 0;                  // Khat, later V
constexpr uint32_t BUF_H = kTileBytes;         // bf16 H_0, later U_0
constexpr uint32_t BUF_D = 2 * kTileBytes;     // q, then the operand E, then the output tile
constexpr uint32_t OFF_SC = 3 * kTileBytes;    // scalars

struct GateScalars {       // per token of a tile, from the gates and the other per-token inputs alone
    float lg[NT];          // log2 gamma_c
    float G2[NT];          // cumulative log2 gate
    float ac[NT];          // G2_c - max(G2_c, -60): exponent correction of clamped tokens
    float zt[NT];          // clamped zeta_c
    float iz[NT];          // 1 / zt_c
    float lam[NT];         // lambda_c as given
    float al[NT];          // alpha_c (alpha-connection)
    float sb[NT];          // sqrt(beta_j) (beta-augmented write)
    float ks[NT];          // row factor of the staged keys: sb_j 2^(-G_j / 2), or sb_j alone when the tile decays below 2^-60
};
struct TileScalars {
    GateScalars g[2];
    float rho2[NT], czb[NT], lz[NT];   // rho^2;  -zt 2 / (L + mu) (0 past the sequence);  lambda / zt
    float part[2][2][NT];              // Frobenius partial sums: [k H_0 k | Gram part][column half][key]
    float carry[2][4];                 // per-warp totals (a, b) of the affine scan
    int stop;
};
constexpr uint32_t SC_BYTES = (sizeof(TileScalars) + 127) / 128 * 128;
constexpr uint32_t SOLVE_SMEM = OFF_SC + SC_BYTES + 1024;   // + slack for the 1024-byte alignment of the base
static_assert(kBlocksPerSM * (SOLVE_SMEM + 1024 + 256) <= 233472, "shared memory budget of two blocks per SM");

// ---- TMEM columns: score accumulator S (P overwrites it in place), residual / output accumulator R
constexpr uint32_t TM_S = 0, TM_R = 128;

enum {
    B_LD_K = 0,    // K tile has landed (TMA)
    B_LD_H,        // H_0 tile
    B_LD_Q,        // q tile
    B_LD_U,        // U_0 tile
    B_LD_V,        // V tile
    B_RDY,         // compute warps -> MMA issuer: operands of the next batch are in place (one arrival per warp)
    B_RDY_ST,      // compute warps -> TMA thread: the output tile is staged
    B_MMA_S,       // tcgen05.commit: score-side batch complete
    B_MMA_R,       // tcgen05.commit: accumulator-side batch complete
    B_GS0, B_GS1,  // gate scalars of buffer 0 / 1 are ready
    B_GF0, B_GF1,  // compute warps -> gate helper: buffer 0 / 1 is free
    B_DRAIN,       // every product is complete (before the tensor memory is given back)
    B_COUNT
};

struct Ctx {
    int tid, l, q, hf, c;         // thread, lane, TMEM lane quadrant, column half, token / TMEM lane
    uint32_t lane_addr, sbase, bars, tmem, abort_addr;
    unsigned char *smem;
};

__device__ __forceinline__ bool aborted(uint32_t abort_addr) {
    int v;
    asm volatile("ld.volatile.shared.b32 %0, [%1];" : "=r"(v) : "r"(abort_addr) : "memory");
    return v != 0;
}
__device__ __forceinline__ void set_abort(uint32_t abort_addr) {
    asm volatile("st.volatile.shared.b32 [%0], %1;" ::"r"(abort_addr), "r"(1) : "memory");
}
// Bounded wait; once any wait of the block has given up every later wait returns at once, so the block runs to its
// end without further delays and reports GKA_ERR_TIMEOUT.
__device__ __forceinline__ void wait_bar(uint32_t bar, uint32_t parity, uint32_t abort_addr) {
    if (aborted(abort_addr)) return;
    if (!mbar_spin_bounded(bar, parity)) set_abort(abort_addr);
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

// Masked score epilogue: S (TMEM, fp32) -> P (packed bf16 pairs, written over the first 16 columns of each 32-column
// block of the scores).  A thread owns token c = 32 q + l and the key blocks kb = 2 hf, 2 hf + 1 (keys 32 kb + i):
// blocks above the diagonal are zero, blocks below it need no mask.  EXACT: per-element factor 2^(ac_c - G_j)
// (strongly decaying tiles, whose keys are not pre-scaled).
template <bool EXACT, bool DIAG, bool KEYF>
__device__ __forceinline__ void p_block(const Ctx &cx, const float *G2kb, const float *kskb, uint32_t taddr, float ac_c) {
#pragma unroll
    for (int piece = 0; piece < 2; ++piece) {
        uint32_t r[16], pk[8];
        TMEM_LD16(taddr + 16 * piece, r);
        tmem_wait_ld();
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i0 = 16 * piece + 2 * u;
            float p0 = __uint_as_float(r[2 * u]), p1 = __uint_as_float(r[2 * u + 1]);
            if (EXACT) {
                p0 *= ex2_fast(fminf(ac_c - G2kb[i0], 126.f));
                p1 *= ex2_fast(fminf(ac_c - G2kb[i0 + 1], 126.f));
            }
            if (KEYF) {                     // the values are not pre-scaled: their row factor rides on the scores
                const float2 f = *reinterpret_cast<const float2 *>(kskb + i0);
                p0 *= f.x;
                p1 *= f.y;
            }
            if (DIAG) {                     // keys i <= l are visible
                p0 = (i0 <= cx.l) ? p0 : 0.f;
                p1 = (i0 + 1 <= cx.l) ? p1 : 0.f;
            }
            pk[u] = pack_bf16(p0, p1);
        }
        TMEM_ST8(taddr + 8 * piece, pk);
    }
}
// keyf: multiply key j's column by ks[j] as well (the pass whose P meets the unscaled V)
template <bool KEYF>
__device__ __forceinline__ void p_epilogue(const Ctx &cx, uint32_t tm_s, const GateScalars *gs, bool exact, float ac_c) {
#pragma unroll
    for (int b2 = 0; b2 < 2; ++b2) {
        const int kb = 2 * cx.hf + b2;
        const uint32_t taddr = tm_s + cx.lane_addr + 32 * kb;
        const float *G2kb = gs->G2 + 32 * kb, *kskb = gs->ks + 32 * kb;
        if (kb > cx.q) {
            uint32_t z[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) z[i] = 0u;
            TMEM_ST8(taddr, z);
            TMEM_ST8(taddr + 8, z);
        } else if (kb == cx.q) {
            if (exact) p_block<true, true, KEYF>(cx, G2kb, kskb, taddr, ac_c);
            else p_block<false, true, KEYF>(cx, G2kb, kskb, taddr, ac_c);
        } else {
            if (exact) p_block<true, false, KEYF>(cx, G2kb, kskb, taddr, ac_c);
            else p_block<false, false, KEYF>(cx, G2kb, kskb, taddr, ac_c);
        }
    }
    tmem_wait_st();
}

// Scale the 128 rows of a bf16 operand tile in place by the per-row factors f[j].
__device__ __forceinline__ void scale_rows(unsigned char *tile, const float *f, int tid) {
#pragma unroll
    for (int i = 0; i < 2048 / CT; ++i) {
        const int qi = tid + CT * i;               // 16-byte group index in the 32 KB tile
        const float fj = f[(qi & 1023) >> 3];      // row of this group
        const uint64_t f2 = f2_pack(fj, fj);
        uint4 v = *reinterpret_cast<const uint4 *>(tile + qi * 16);
        uint32_t *pv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            float lo, hi;
            f2_unpack(f2_mul(f2_pack(bf16_lo(pv[u]), bf16_hi(pv[u])), f2), lo, hi);
            pv[u] = pack_bf16(lo, hi);
        }
        *reinterpret_cast<uint4 *>(tile + qi * 16) = v;
    }
}

// Inclusive scan over the tile's 128 tokens (threads 0..127 = warps 0..3, one token each) of the affine maps
// s -> a s + b, composed in token order; returns the map's value at `seed`.
__device__ __forceinline__ float affine_scan(const Ctx &cx, TileScalars *sc, float a, float b, float seed) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float pa = __shfl_up_sync(0xffffffffu, a, o), pb = __shfl_up_sync(0xffffffffu, b, o);
        if (cx.l >= o) {
            b = fmaf(a, pb, b);
            a *= pa;
        }
    }
    if (cx.l == 31) {
        sc->carry[0][cx.q] = a;
        sc->carry[1][cx.q] = b;
    }
    asm volatile("bar.sync 2, 128;" ::: "memory");
    float s = seed;
    for (int w = 0; w < cx.q; ++w) s = fmaf(sc->carry[0][w], s, sc->carry[1][w]);
    return fmaf(a, s, b);
}

// Batches of products the issuing thread runs, one per arrival phase of B_RDY, in this order per tile:
// FROB, then n_iter times (ITER1, ITER2), then (unless the solve itself is the result) OUT_S, OUT_O.
__device__ __forceinline__ void issue_batch(int op, uint32_t base14, uint32_t tm, uint32_t bars) {
    const uint32_t kb = base14 + (BUF_K >> 4), hb = base14 + (BUF_H >> 4), db = base14 + (BUF_D >> 4);
    const uint32_t tm_S = tm + TM_S, tm_R = tm + TM_R;
    switch (op) {
        case 0:   // FROB: Gram matrix Khat Khat^T and Khat H_0
            mma8_kk<0>(tm_S, kb, kb, kIdescKK);
            mma8_kk<0>(tm_R, kb, hb, kIdescKK);
            mma_commit(bars + 8 * B_MMA_S);
            break;
        case 1:   // ITER1: S = E Khat^T, R += E H_0^T (the second runs under the masked-score epilogue)
            mma8_kk<0>(tm_S, db, kb, kIdescKK);
            mma_commit(bars + 8 * B_MMA_S);
            mma8_kk<1>(tm_R, db, hb, kIdescKK);
            break;
        case 2:   // ITER2: R += P Khat
            mma8_pm(tm_R, tm_S, kb, kIdescPM);
            mma_commit(bars + 8 * B_MMA_R);
            break;
        case 3:   // OUT_S: scores of the final iterate, S = X_hi Khat^T + X_lo Khat^T (X_lo sits in the H_0 buffer)
            mma8_kk<0>(tm_S, db, kb, kIdescKK);
            mma8_kk<1>(tm_S, hb, kb, kIdescKK);
            mma_commit(bars + 8 * B_MMA_S);
            break;
        default:  // OUT_O: O = X_hi U_0^T + P V
            mma8_kk<0>(tm_R, db, hb, kIdescKK);
            mma8_pm(tm_R, tm_S, kb, kIdescPM);
            mma_commit(bars + 8 * B_MMA_R);
            break;
    }
}

template <bool EXTRA>
__global__ void __launch_bounds__(kThreadsSolve, kBlocksPerSM)
fwd_tc_solve_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmO,
                    const __grid_constant__ CUtensorMap tmS, FwdArgs a, long long ntiles) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_bars[B_COUNT];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    unsigned char *smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    const int tid = threadIdx.x;
    const uint32_t bars = smem_u32(&s_bars[0]);
    const uint32_t abort_addr = smem_u32(&s_abort);

    if (tid == 0) {
        s_abort = 0;
        for (int i = 0; i < B_COUNT; ++i) {
            const int count = (i == B_RDY || i == B_RDY_ST || i == B_GF0 || i == B_GF1) ? NW : 1;
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bars + 8 * i), "r"(count));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(smem_u32(&s_tmem_base))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = s_tmem_base;
    const uint32_t sbase = smem_u32(smem);
    TileScalars *const sc = reinterpret_cast<TileScalars *>(smem + OFF_SC);

    // this block's tiles: a contiguous range
    const long long t_lo = (ntiles * blockIdx.x) / gridDim.x, t_hi = (ntiles * (blockIdx.x + 1)) / gridDim.x;
    const int n_mine = (int)(t_hi - t_lo);
    const bool solve_only = EXTRA && a.solve_only != 0;   // the result is the solve itself: no V, no U, no output product
    const float *const beta_p = EXTRA ? a.beta : nullptr;
    const float *const alpha_p = EXTRA ? a.alpha : nullptr;
    const bool mix = alpha_p != nullptr && !solve_only;   // alpha-connection: the read uses alpha x + (1 - alpha) q

    if (tid >= CT) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsHelper));
        const int hw = (tid - CT) >> 5, lane = tid & 31;
        if (hw == 0) {
            // ================= gate scalars of every tile, one tile ahead of the compute warps =================
            for (int k = 0; k < n_mine; ++k) {
                if (k >= 2) wait_bar(bars + 8 * (B_GF0 + (k & 1)), (uint32_t)(((k - 2) >> 1) & 1), abort_addr);
                const TileInfo ti = tile_info(a, t_lo + k);
                GateScalars *g = &sc->g[k & 1];
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
                    g->sb[cc] = sqrtf(fmaxf(bv, 0.f));
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
                if (lane == 0) mbar_arrive(bars + 8 * (B_GS0 + (k & 1)));
            }
        } else if (hw == 1) {
            // ================= TMA: loads of every tile's K, H_0, q; stores of the output tiles =================
            if (lane == 0) {
                auto load_k = [&](int k) {
                    const TileInfo ti = tile_info(a, t_lo + k);
                    mbar_expect_tx(bars + 8 * B_LD_K, 32768u);
                    tma_load_tile3(&tmK, sbase + BUF_K, bars + 8 * B_LD_K, ti.h * D, ti.n * NT, ti.b);
                };
                auto load_h = [&](int k) {
                    mbar_expect_tx(bars + 8 * B_LD_H, 32768u);
                    tma_load_tile2(&tmS, sbase + BUF_H, bars + 8 * B_LD_H, (int)((t_lo + k) * 256));
                };
                auto load_q = [&](int k) {
                    const TileInfo ti = tile_info(a, t_lo + k);
                    mbar_expect_tx(bars + 8 * B_LD_Q, 32768u);
                    tma_load_tile3(&tmQ, sbase + BUF_D, bars + 8 * B_LD_Q, ti.h * D, ti.n * NT, ti.b);
                };
                // the inputs do not depend on the state kernel; its per-tile states do
                if (n_mine > 0) {
                    load_q(0);
                    load_k(0);
                }
                asm volatile("griddepcontrol.wait;" ::: "memory");
                if (n_mine > 0) load_h(0);
                // The result tile is staged in the H_0 / U_0 buffer (the solve alone: in the operand buffer).  The other
                // two buffers of the next tile are loaded by a compute thread as soon as the last product is complete;
                // the staging buffer's next content follows once the store has read it.
                const uint32_t stage_buf = solve_only ? BUF_D : BUF_H;
                for (int k = 0; k < n_mine; ++k) {
                    wait_bar(bars + 8 * B_RDY_ST, (uint32_t)(k & 1), abort_addr);
                    const TileInfo ti = tile_info(a, t_lo + k);
                    for (int hf = 0; hf < 2; ++hf)     // rows past the sequence are clipped
                        asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];" ::
                                         "l"(reinterpret_cast<uint64_t>(&tmO)), "r"(ti.h * D + 64 * hf), "r"(ti.n * NT),
                                     "r"(ti.b), "r"(sbase + stage_buf + 16384 * hf)
                                     : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    const bool more = k + 1 < n_mine && !aborted(abort_addr);
                    if (more && solve_only) {
                        load_k(k + 1);
                        load_h(k + 1);
                    }
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the staged tile has been read
                    if (more) {
                        if (solve_only) load_q(k + 1);
                        else load_h(k + 1);
                    }
                }
                asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // output stores are complete
            }
        } else if (hw == 2) {
            // ================================ MMA issuing thread ================================
            if (lane == 0) {
                const uint32_t base14 = (sbase >> 4) & 0x3FFF;
                uint32_t n_rdy = 0;
                auto batch = [&](int op, int k) {
                    wait_bar(bars + 8 * B_RDY, n_rdy & 1u, abort_addr);
                    ++n_rdy;
                    // the first batch also needs the H_0 tile, the last one the U_0 tile (TMA)
                    if (op == 0) wait_bar(bars + 8 * B_LD_H, (uint32_t)(k & 1), abort_addr);
                    if (op == 4) {
                        wait_bar(bars + 8 * B_LD_U, (uint32_t)(k & 1), abort_addr);
                        wait_bar(bars + 8 * B_LD_V, (uint32_t)(k & 1), abort_addr);
                    }
                    fence_after();
                    issue_batch(op, base14, tmem, bars);
                };
                for (int k = 0; k < n_mine; ++k) {
                    batch(0, k);
                    for (int it = 0; it < a.n_iter; ++it) {
                        batch(1, k);
                        batch(2, k);
                    }
                    if (!solve_only) {
                        batch(3, k);
                        batch(4, k);
                    }
                }
                // every product is complete before the block gives its tensor memory back
                mma_commit(bars + 8 * B_DRAIN);
                if (!mbar_spin_bounded(bars + 8 * B_DRAIN, 0u)) set_abort(abort_addr);
            }
        }
    } else {
        // ================================= compute threads =================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsCompute));
        Ctx cx;
        cx.tid = tid;
        cx.l = tid & 31;
        cx.q = (tid >> 5) & 3;
        cx.hf = tid >> 7;
        cx.c = 32 * cx.q + cx.l;
        cx.lane_addr = (uint32_t)(32 * cx.q) << 16;
        cx.smem = smem;
        cx.sbase = sbase;
        cx.bars = bars;
        cx.tmem = tmem;
        cx.abort_addr = abort_addr;
        const int c = cx.c, hf = cx.hf, l = cx.l;
        const bool adaptive = (a.flags & GKA_FLAG_ADAPTIVE_LAMBDA) != 0;
        const uint32_t tm_s = tmem + TM_S, tm_r = tmem + TM_R;
        unsigned char *const bufk = smem + BUF_K, *const bufh = smem + BUF_H, *const bufd = smem + BUF_D;
        // the per-tile states and norms come from the state kernel
        asm volatile("griddepcontrol.wait;" ::: "memory");

        uint64_t xs[32];                    // -zt_c x_c, this thread's 64 channels as fp32 pairs
        uint32_t n_s = 0, n_r = 0, n_q = 0;   // completed phases of MMA_S, MMA_R, LD_Q
        auto wait_s = [&]() { wait_bar(bars + 8 * B_MMA_S, n_s & 1u, abort_addr); ++n_s; fence_after(); };
        auto wait_r = [&]() { wait_bar(bars + 8 * B_MMA_R, n_r & 1u, abort_addr); ++n_r; fence_after(); };
        auto arrive_rdy = [&]() { warp_arrive(bars + 8 * B_RDY, l); };
        // stage -xs (times `scale`) as bf16: its leading part, or the remainder after the leading part
        auto stage_x = [&](unsigned char *dst, bool lo, float scale) {
#pragma unroll
            for (int g8 = 0; g8 < 8; ++g8) {
                uint32_t pk[4];
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
                *reinterpret_cast<uint4 *>(dst + tile_off(c, 8 * hf + g8)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
        };

        for (int k = 0; k < n_mine; ++k) {
            const long long tile = t_lo + k;
            const GateScalars *const gs = &sc->g[k & 1];
            const TileInfo ti = tile_info(a, tile);
            const bool valid = c < ti.ntok;
            // ||H_0||_F^2 of the tile (state kernel): fetched now, used by the scan
            const float hh = tid < NT ? ldg_stream_f32(a.tile_hh + tile) : 0.f;
            // ---- gate scalars (helper warp) and the K, H_0 tiles (TMA) of this tile
            wait_bar(bars + 8 * (B_GS0 + (k & 1)), (uint32_t)((k >> 1) & 1), abort_addr);
            wait_bar(bars + 8 * B_LD_K, (uint32_t)(k & 1), abort_addr);
            const bool exact = gs->G2[ti.ntok - 1] < -60.f;     // the tile decays below 2^-60: per-element factors
            scale_rows(bufk, gs->ks, tid);
            fence_async_smem();
            arrive_rdy();                                        // -> FROB
            wait_s();
            // ---- chunk-wise Frobenius norms: per key, k_j^T H_0 k_j and the decayed squared Gram entries of the
            // earlier keys.  Thread = (key j = c, 64 columns).
            {
                float kh = 0.f, gsum = 0.f;
#pragma unroll
                for (int piece = 0; piece < 2; ++piece) {
                    uint32_t r[32];
                    TMEM_LD32(tm_r + cx.lane_addr + 64 * hf + 32 * piece, r);
                    uint4 kv[4];
#pragma unroll
                    for (int h4 = 0; h4 < 4; ++h4) kv[h4] = *reinterpret_cast<const uint4 *>(bufk + tile_off(c, 8 * hf + 4 * piece + h4));
                    tmem_wait_ld();
#pragma unroll
                    for (int h4 = 0; h4 < 4; ++h4) {
                        const uint32_t *pk = reinterpret_cast<const uint32_t *>(&kv[h4]);
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            kh = fmaf(__uint_as_float(r[8 * h4 + 2 * u]), bf16_lo(pk[u]), kh);
                            kh = fmaf(__uint_as_float(r[8 * h4 + 2 * u + 1]), bf16_hi(pk[u]), kh);
                        }
                    }
                }
                const float G2j = gs->G2[c];
#pragma unroll
                for (int b2 = 0; b2 < 2; ++b2) {
                    const int kb = 2 * hf + b2;
                    if (kb > cx.q) continue;
                    const int lim = (kb == cx.q) ? l : 32;   // keys i < lim come earlier, i == lim is the key itself
                    float gs2 = 0.f, gd = 0.f;
                    uint32_t r[32];
                    TMEM_LD32(tm_s + cx.lane_addr + 32 * kb, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int ii = 0; ii < 32; ++ii) {
                        const float g = __uint_as_float(r[ii]);
                        const float g2 = g * g;
                        if (ii == lim) gd = g2;
                        if (!exact) gs2 += (ii < lim) ? g2 : 0.f;
                        else if (ii < lim) gs2 = fmaf(ex2_fast(G2j - gs->G2[32 * kb + ii]), g2, gs2);
                    }
                    gsum += 2.f * gs2 + gd;
                }
                sc->part[0][hf][c] = kh;
                sc->part[1][hf][c] = gsum;
            }
            fence_before();
            if (tid == 0) sc->stop = aborted(abort_addr) ? 1 : 0;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            // ---- f_c by an affine scan (s_c = gamma_c^2 s_{c-1} + d_c, s_{-1} = ||H_0||^2), Chebyshev set-up
            if (tid < NT) {
                const float kh = sc->part[0][0][c] + sc->part[0][1][c];
                const float gsum = sc->part[1][0][c] + sc->part[1][1][c];
                const float G2c = gs->G2[c];
                // pre-scaled keys: both sums carry 2^(-2 G_c); plain keys: k H_0 k carries zeta_c
                const float dc = exact ? fmaf(2.f * ex2_fast(G2c), kh, gsum) : ex2_fast(2.f * G2c) * fmaf(2.f, kh, gsum);
                const float s = affine_scan(cx, sc, ex2_fast(2.f * gs->lg[c]), dc, hh);
                const float fc = sqrtf(fmaxf(s, 0.f));
                float lamc = gs->lam[c];
                if (adaptive) lamc *= fc;
                const float Lpm = fc + 2.f * lamc;
                const float iL = 1.f / Lpm;
                const float rho = fc * iL;
                sc->rho2[c] = rho * rho;
                sc->czb[c] = valid ? -gs->zt[c] * (2.f * iL) : 0.f;
                sc->lz[c] = lamc * gs->iz[c];
                if (a.fro_out && valid) a.fro_out[ti.tok0 + (size_t)c * a.heads] = fc;
            }
            wait_bar(bars + 8 * B_LD_Q, n_q & 1u, abort_addr);   // q tile has landed
            ++n_q;
            asm volatile("bar.sync 1, 256;" ::: "memory");       // the set-up values are published
            if (sc->stop) break;                                 // the same decision in every thread
            const float rho2 = sc->rho2[c], czb = sc->czb[c], lz = sc->lz[c];
            // ---- x_0: R = q, E_0 = czb q (in place of q), xs = E_0
#pragma unroll
            for (int g16 = 0; g16 < 4; ++g16) {
                uint32_t rr[16];
#pragma unroll
                for (int h2 = 0; h2 < 2; ++h2) {
                    const int g8 = 2 * g16 + h2;
                    const uint4 qv = *reinterpret_cast<const uint4 *>(bufd + tile_off(c, 8 * hf + g8));
                    const uint32_t *qq = reinterpret_cast<const uint32_t *>(&qv);
                    uint32_t pk[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float qa = bf16_lo(qq[u]), qb = bf16_hi(qq[u]);
                        rr[8 * h2 + 2 * u] = __float_as_uint(qa);
                        rr[8 * h2 + 2 * u + 1] = __float_as_uint(qb);
                        pk[u] = pack_bf16(czb * qa, czb * qb);
                        xs[4 * g8 + u] = f2_pack(bf16_lo(pk[u]), bf16_hi(pk[u]));
                    }
                    *reinterpret_cast<uint4 *>(bufd + tile_off(c, 8 * hf + g8)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
                TMEM_ST16(tm_r + cx.lane_addr + 64 * hf + 16 * g16, rr);
            }
            tmem_wait_st();
            // ---- Algorithm 1
            float omega = 2.f;
            if (a.n_iter > 0) {
                fence_async_smem();
                fence_before();
                arrive_rdy();                                    // -> ITER1
            }
            for (int it = 0; it < a.n_iter; ++it) {
                const bool last = it + 1 == a.n_iter;
                omega = 4.f / (4.f - rho2 * omega);              // weight schedule
                const float beta = omega - 1.f, cz = czb * omega;
                wait_s();
                p_epilogue<false>(cx, tm_s, gs, exact, gs->ac[c]);
                fence_before();
                arrive_rdy();                                    // -> ITER2
                const uint64_t beta2 = f2_pack(beta, beta), cz2 = f2_pack(cz, cz), lz2 = f2_pack(lz, lz);
                wait_r();
                // e_new = beta e_old + cz (R + lz xs); xs += e_new (as rounded for the operand, unless last).  Eight
                // channels at a time; the next group's loads are in flight while a group is computed.
                {
                    uint32_t ra[8], rb[8];
                    uint4 eva, evb;
                    TMEM_LD8(tm_r + cx.lane_addr + 64 * hf, ra);
                    eva = *reinterpret_cast<const uint4 *>(bufd + tile_off(c, 8 * hf));
                    tmem_wait_ld();
#pragma unroll
                    for (int g8 = 0; g8 < 8; ++g8) {
                        uint32_t(&r)[8] = (g8 & 1) ? rb : ra;
                        uint32_t(&rn)[8] = (g8 & 1) ? ra : rb;
                        uint4 &ev = (g8 & 1) ? evb : eva;
                        uint4 &evn = (g8 & 1) ? eva : evb;
                        if (g8 < 7) {
                            TMEM_LD8(tm_r + cx.lane_addr + 64 * hf + 8 * (g8 + 1), rn);
                            evn = *reinterpret_cast<const uint4 *>(bufd + tile_off(c, 8 * hf + g8 + 1));
                        }
                        const uint32_t *ee = reinterpret_cast<const uint32_t *>(&ev);
                        uint32_t pk[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int i = 4 * g8 + u;
                            const uint64_t res = f2_fma(lz2, xs[i], f2_pack(__uint_as_float(r[2 * u]), __uint_as_float(r[2 * u + 1])));
                            const uint64_t en = f2_fma(cz2, res, f2_mul(beta2, f2_pack(bf16_lo(ee[u]), bf16_hi(ee[u]))));
                            float ea, eb;
                            f2_unpack(en, ea, eb);
                            pk[u] = pack_bf16(ea, eb);
                            xs[i] = f2_add(xs[i], last ? en : f2_pack(bf16_lo(pk[u]), bf16_hi(pk[u])));
                        }
                        if (!last) {
                            *reinterpret_cast<uint4 *>(bufd + tile_off(c, 8 * hf + g8)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                            if (g8 == 7) {
                                fence_async_smem();
                                fence_before();     // the accumulator R has been read completely
                                arrive_rdy();       // -> ITER1
                            }
                        }
                        if (g8 < 7) tmem_wait_ld();
                    }
                }
            }
            // ---- final iterate
            if (solve_only) {
                // the solve is the result: x_c = -xs / zt_c as bf16, stored by TMA
                stage_x(bufd, false, gs->iz[c]);
                fence_async_smem();
                warp_arrive(bars + 8 * (B_GF0 + (k & 1)), l);
                warp_arrive(bars + 8 * B_RDY_ST, l);
                continue;
            }
            if (mix) {
                // alpha-connection (Section 4.3): the read uses alpha x + (1 - alpha) q; q comes back into the H_0
                // buffer, which no product reads any more
                if (tid == 0) {
                    mbar_expect_tx(bars + 8 * B_LD_Q, 32768u);
                    tma_load_tile3(&tmQ, sbase + BUF_H, bars + 8 * B_LD_Q, ti.h * D, ti.n * NT, ti.b);
                }
                wait_bar(bars + 8 * B_LD_Q, n_q & 1u, abort_addr);
                ++n_q;
                const float alc = gs->al[c], nzt = valid ? -gs->zt[c] : 0.f;
#pragma unroll
                for (int g8 = 0; g8 < 8; ++g8) {
                    const uint4 qv = *reinterpret_cast<const uint4 *>(bufh + tile_off(c, 8 * hf + g8));
                    const uint32_t *qq = reinterpret_cast<const uint32_t *>(&qv);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        float xa, xb;
                        f2_unpack(xs[4 * g8 + u], xa, xb);
                        const float qa = nzt * bf16_lo(qq[u]), qb = nzt * bf16_hi(qq[u]);
                        xs[4 * g8 + u] = f2_pack(fmaf(alc, xa - qa, qa), fmaf(alc, xb - qb, qb));
                    }
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");   // every thread has read q: U_0 may overwrite it
            }
            // The read uses the final iterate as two bf16 terms in the score product (the recent keys resolve directions
            // of x that one bf16 rounding would lose); the second term takes the H_0 buffer, which no product reads
            // any more.
            stage_x(bufd, false, 1.f);
            stage_x(bufh, true, 1.f);
            fence_async_smem();
            fence_before();
            arrive_rdy();                                        // -> OUT_S
            wait_s();
            if (tid == 0) {               // the keys and the second term are no longer needed: V and U_0 take their buffers
                mbar_expect_tx(bars + 8 * B_LD_V, 32768u);
                tma_load_tile3(&tmV, sbase + BUF_K, bars + 8 * B_LD_V, ti.h * D, ti.n * NT, ti.b);
                mbar_expect_tx(bars + 8 * B_LD_U, 32768u);
                tma_load_tile2(&tmS, sbase + BUF_H, bars + 8 * B_LD_U, (int)(tile * 256 + 128));
            }
            // the values stay as loaded: their row factor sqrt(beta_j) 2^(-G_j / 2) rides on the masked scores
            p_epilogue<true>(cx, tm_s, gs, exact, gs->ac[c]);
            fence_before();
            arrive_rdy();                                        // -> OUT_O
            wait_r();
            // every product of the tile is complete: the next tile's K and q can come in (H_0 follows the store)
            if (tid == 0 && k + 1 < n_mine) {
                const TileInfo tn = tile_info(a, tile + 1);
                mbar_expect_tx(bars + 8 * B_LD_K, 32768u);
                tma_load_tile3(&tmK, sbase + BUF_K, bars + 8 * B_LD_K, tn.h * D, tn.n * NT, tn.b);
                mbar_expect_tx(bars + 8 * B_LD_Q, 32768u);
                tma_load_tile3(&tmQ, sbase + BUF_D, bars + 8 * B_LD_Q, tn.h * D, tn.n * NT, tn.b);
            }
            // O as bf16 into the U_0 buffer (no product reads it any more), stored by TMA
#pragma unroll
            for (int piece = 0; piece < 4; ++piece) {
                uint32_t r[16];
                TMEM_LD16(tm_r + cx.lane_addr + 64 * hf + 16 * piece, r);
                tmem_wait_ld();
                uint32_t pk[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) pk[u] = pack_bf16(__uint_as_float(r[2 * u]), __uint_as_float(r[2 * u + 1]));
                *reinterpret_cast<uint4 *>(bufh + tile_off(c, 8 * hf + 2 * piece)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                *reinterpret_cast<uint4 *>(bufh + tile_off(c, 8 * hf + 2 * piece + 1)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
            }
            fence_async_smem();
            fence_before();
            warp_arrive(bars + 8 * (B_GF0 + (k & 1)), l);
            warp_arrive(bars + 8 * B_RDY_ST, l);
        }
        if (aborted(abort_addr)) set_abort(abort_addr);
    }

    fence_before();
    __syncthreads();
    if (s_abort != 0) {
        // a wait gave up: leave time for copies still in flight before the shared memory is given back
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        if (tid == 0 && a.device_status) atomicExch(a.device_status, (int)GKA_ERR_TIMEOUT);
    }
    if (tid < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
}

}  // namespace

cudaError_t launch_fwd_solve(const FwdArgs &a, cudaStream_t stream) {
    alignas(64) CUtensorMap tmK, tmV, tmQ, tmO, tmS;
    const int cols = a.heads * D;
    const long long ntiles = a.plan.NC;
    if (!make_tile_map(&tmK, a.k, a.B, a.T, cols, NT) || !make_tile_map(&tmV, a.v, a.B, a.T, cols, NT) ||
        !make_tile_map(&tmQ, a.q, a.B, a.T, cols, NT) || !make_tile_map(&tmO, a.out, a.B, a.T, cols, NT) ||
        !make_state_map(&tmS, a.tile_hu, (unsigned long long)ntiles * 256ull))
        return cudaErrorInvalidValue;
    const bool extra = a.beta != nullptr || a.alpha != nullptr || a.solve_only != 0;
    auto kernel = extra ? fwd_tc_solve_kernel<true> : fwd_tc_solve_kernel<false>;
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SOLVE_SMEM);
    if (err != cudaSuccess) return err;
    int dev = 0, sms = 0;
    if ((err = cudaGetDevice(&dev)) != cudaSuccess) return err;
    if ((err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return err;
    const long long want = (long long)kBlocksPerSM * sms;
    if (a.ev_start) cudaEventRecord(a.ev_start, stream);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(ntiles < want ? ntiles : want));
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
