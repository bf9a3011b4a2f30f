// tcgen05 / TMEM solve kernel of the chunk-wise GKA forward (bf16 operands, fp32 accumulation) for sm_100a.
//
// Input: for every tile of 128 consecutive tokens of a sequence, the bf16 copies of the tile-initial states
// H_0, U_0 and ||H_0||_F^2 (written by the state kernel, gka_tc_state.cu).  Tiles are independent problems; a
// persistent thread block per SM keeps TWO of them in flight ("chains"), so that the tensor-core products of one
// run under the CUDA-core epilogues of the other.  A tile puts one token on each TMEM lane; every product of the
// chunk-wise form (Section 4.2.1; Algorithm 1 on the whole tile) is an M = 128 tile.
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
// Warp roles: 16 compute warps (warp quadrant q = TMEM lanes 32 q .. 32 q + 31, column quarter cq = 32 of the 128
// columns: a thread holds one token's 32 channels of both chains' iterates in registers); one warp prepares the
// gate scalars one tile ahead; one warp issues TMA loads and stores; one thread issues every tcgen05.mma.  The
// compute warps hand work over through mbarriers (one arrival per warp) and wait for tcgen05.commit.
#include <cuda.h>

#include "gka_common.cuh"
#include "gka_tc_mma.cuh"

namespace gka {
namespace {

using namespace tcu;

constexpr int D = 128;
constexpr int NT = kTile;                  // tokens per tile: one per TMEM lane
constexpr int CT = 512;                    // compute threads
constexpr int kThreadsSolve = CT + 128;    // + helper warpgroup: gate scalars, TMA, MMA issue
constexpr int kRegsCompute = 112, kRegsHelper = 32;   // register split after setmaxnreg (launch: 96 each)
static_assert(CT * kRegsCompute + 128 * kRegsHelper <= kThreadsSolve * 96, "register split exceeds the launch allocation");

// ---- shared memory map (bytes; operand buffers 1024-byte aligned).  Per chain three operand tiles:
constexpr uint32_t CH_STRIDE = 3 * kTileBytes;
constexpr uint32_t BUF_K = 0;                  // Khat, later Vhat
constexpr uint32_t BUF_H = kTileBytes;         // bf16 H_0, later U_0
constexpr uint32_t BUF_D = 2 * kTileBytes;     // q, then the operand E, then the output tile
constexpr uint32_t OFF_SC = 2 * CH_STRIDE;     // scalars

struct GateScalars {       // per token of a tile, from the gates and the other per-token inputs alone
    float lg[NT];          // log2 gamma_c
    float G2[NT];          // cumulative log2 gate
    float ac[NT];          // G2_c - max(G2_c, -60): exponent correction of clamped tokens
    float zt[NT];          // clamped zeta_c
    float iz[NT];          // 1 / zt_c
    float lam[NT];         // lambda_c as given
    float al[NT];          // alpha_c (alpha-connection)
    float sb[NT];          // sqrt(beta_j) (beta-augmented write)
};
struct ChainScalars {
    GateScalars g[2];
    float rho2[NT], czb[NT], lz[NT];   // rho^2;  -zt 2 / (L + mu) (0 past the sequence);  lambda / zt
    float part[2][4][NT];              // Frobenius partial sums: [k H_0 k | Gram part][column quarter][key]
    float carry[2][4];                 // per-warp totals (a, b) of the affine scan
    int stop;
    int exact;                         // the tile decays below 2^-60: unscaled keys, per-element factors
};
constexpr uint32_t SC_BYTES = 2 * ((sizeof(ChainScalars) + 127) / 128 * 128);
constexpr uint32_t SOLVE_SMEM = OFF_SC + SC_BYTES + 1024;   // + slack for the 1024-byte alignment of the base
static_assert(SOLVE_SMEM <= 232448 - 512, "shared memory budget");

// ---- TMEM columns per chain: score accumulator S (P overwrites it in place), residual / output accumulator R
constexpr uint32_t TM_CHAIN = 256, TM_S = 0, TM_R = 128;

// ---- mbarriers, per chain
enum {
    B_LD_KH = 0,   // K and H_0 tiles have landed (TMA)
    B_LD_Q,        // q tile
    B_LD_U,        // U_0 tile
    B_LD_V,        // V tile
    B_RDY,         // compute warps -> MMA issuer: operands of the next batch are in place (16 arrivals)
    B_RDY_ST,      // compute warps -> TMA warp: the output tile is staged (16 arrivals)
    B_MMA_S,       // tcgen05.commit: score-side batch complete
    B_MMA_R,       // tcgen05.commit: accumulator-side batch complete
    B_GS0, B_GS1,  // gate scalars of buffer 0 / 1 are ready
    B_GF0, B_GF1,  // compute warps -> gate helper: buffer 0 / 1 is free (16 arrivals)
    B_PER_CHAIN
};

struct Ctx {
    int tid, l, q, cq, c;
    uint32_t lane_addr, sbase, bars, tmem, abort_addr;
    unsigned char *smem;
};

__device__ __forceinline__ bool aborted(uint32_t abort_addr) {
    int v;
    asm volatile("ld.volatile.shared.b32 %0, [%1];" : "=r"(v) : "r"(abort_addr) : "memory");
    return v != 0;
}
// Bounded wait; once any wait of the block has given up every later wait returns at once, so the block runs to its
// end without further delays and reports GKA_ERR_TIMEOUT.
__device__ __forceinline__ void wait_bar(uint32_t bar, uint32_t parity, uint32_t abort_addr) {
    if (aborted(abort_addr)) return;
    if (!mbar_spin_bounded(bar, parity)) asm volatile("st.volatile.shared.b32 [%0], %1;" ::"r"(abort_addr), "r"(1) : "memory");
}
__device__ __forceinline__ uint32_t chain_bar(uint32_t bars, int ch, int which) { return bars + 8 * (ch * B_PER_CHAIN + which); }

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

// Masked score epilogue: S (TMEM, fp32) -> P (packed bf16 pairs, written over the first 16 of this thread's own 32
// score columns).  Keys j = 32 cq + i, token c = 32 q + l: blocks above the diagonal are zero, blocks below it need
// no mask.  EXACT: per-element factor 2^(ac_c - G_j) (strongly decaying tiles, whose keys are not pre-scaled).
template <bool EXACT, bool DIAG>
__device__ __forceinline__ void p_block(const Ctx &cx, const float *G2, uint32_t taddr, float ac_c) {
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
                p0 *= ex2_fast(fminf(ac_c - G2[32 * cx.cq + i0], 126.f));
                p1 *= ex2_fast(fminf(ac_c - G2[32 * cx.cq + i0 + 1], 126.f));
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
__device__ __forceinline__ void p_epilogue(const Ctx &cx, uint32_t tm_s, const float *G2, bool exact, float ac_c) {
    const uint32_t taddr = tm_s + cx.lane_addr + 32 * cx.cq;
    if (cx.cq > cx.q) {
        uint32_t z[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) z[i] = 0u;
        TMEM_ST8(taddr, z);
        TMEM_ST8(taddr + 8, z);
    } else if (cx.cq == cx.q) {
        if (exact) p_block<true, true>(cx, G2, taddr, ac_c);
        else p_block<false, true>(cx, G2, taddr, ac_c);
    } else {
        if (exact) p_block<true, false>(cx, G2, taddr, ac_c);
        else p_block<false, false>(cx, G2, taddr, ac_c);
    }
    tmem_wait_st();
}

// Scale the 128 rows of a bf16 operand tile in place: row j by sb_j 2^(-G_j / 2), or by sb_j alone (exact mode).
__device__ __forceinline__ void scale_rows(unsigned char *tile, const GateScalars *gs, bool exact, int tid) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int qi = tid + CT * i;               // 16-byte group index in the 32 KB tile
        const int j = (qi & 1023) >> 3;            // row of this group
        const float f = exact ? gs->sb[j] : gs->sb[j] * ex2_fast(-0.5f * gs->G2[j]);
        uint4 v = *reinterpret_cast<const uint4 *>(tile + qi * 16);
        uint32_t *pv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
        for (int u = 0; u < 4; ++u) pv[u] = pack_bf16(bf16_lo(pv[u]) * f, bf16_hi(pv[u]) * f);
        *reinterpret_cast<uint4 *>(tile + qi * 16) = v;
    }
}

// Inclusive scan over the tile's 128 tokens (threads 0..127 = warps 0..3, one token each) of the affine maps
// s -> a s + b, composed in token order; returns the map's value at `seed`.
__device__ __forceinline__ float affine_scan(const Ctx &cx, ChainScalars *cs, float a, float b, float seed) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float pa = __shfl_up_sync(0xffffffffu, a, o), pb = __shfl_up_sync(0xffffffffu, b, o);
        if (cx.l >= o) {
            b = fmaf(a, pb, b);
            a *= pa;
        }
    }
    if (cx.l == 31) {
        cs->carry[0][cx.q] = a;
        cs->carry[1][cx.q] = b;
    }
    asm volatile("bar.sync 2, 128;" ::: "memory");
    float s = seed;
    for (int w = 0; w < cx.q; ++w) s = fmaf(cs->carry[0][w], s, cs->carry[1][w]);
    return fmaf(a, s, b);
}

enum { PH_SETUP_A = 0, PH_SETUP_B, PH_P, PH_X, PH_OUT2, PH_OUT3, PH_OUT4, PH_DONE };

// Batches of products the issuing thread runs, one per arrival phase of B_RDY, in this order per tile:
// FROB, then n_iter times (ITER1, ITER2), then (unless the solve itself is the result) OUT_HI, OUT_LO, OUT_PV.
__device__ __forceinline__ void issue_batch(int op, uint32_t cb14, uint32_t tm, uint32_t bars, int ch, uint32_t ph_ld_u,
                                            uint32_t abort_addr) {
    const uint32_t kb = cb14 + (BUF_K >> 4), hb = cb14 + (BUF_H >> 4), db = cb14 + (BUF_D >> 4);
    const uint32_t tm_S = tm + TM_S, tm_R = tm + TM_R;
    switch (op) {
        case 0:   // FROB: Gram matrix Khat Khat^T and Khat H_0
            mma8_kk<0>(tm_S, kb, kb, kIdescKK);
            mma8_kk<0>(tm_R, kb, hb, kIdescKK);
            mma_commit(chain_bar(bars, ch, B_MMA_S));
            break;
        case 1:   // ITER1: S = E Khat^T, R += E H_0^T (the second runs under the masked-score epilogue)
            mma8_kk<0>(tm_S, db, kb, kIdescKK);
            mma_commit(chain_bar(bars, ch, B_MMA_S));
            mma8_kk<1>(tm_R, db, hb, kIdescKK);
            break;
        case 2:   // ITER2: R += P Khat
            mma8_pm(tm_R, tm_S, kb, kIdescPM);
            mma_commit(chain_bar(bars, ch, B_MMA_R));
            break;
        case 3:   // OUT_HI: S = X_hi Khat^T, O = X_hi U_0^T
            mma8_kk<0>(tm_S, db, kb, kIdescKK);
            wait_bar(chain_bar(bars, ch, B_LD_U), ph_ld_u, abort_addr);
            mma8_kk<0>(tm_R, db, hb, kIdescKK);
            mma_commit(chain_bar(bars, ch, B_MMA_S));
            break;
        case 4:   // OUT_LO: S += X_lo Khat^T, O += X_lo U_0^T
            mma8_kk<1>(tm_S, db, kb, kIdescKK);
            mma8_kk<1>(tm_R, db, hb, kIdescKK);
            mma_commit(chain_bar(bars, ch, B_MMA_S));
            break;
        default:  // OUT_PV: O += P Vhat
            mma8_pm(tm_R, tm_S, kb, kIdescPM);
            mma_commit(chain_bar(bars, ch, B_MMA_R));
            break;
    }
}

template <bool EXTRA>
__global__ void __launch_bounds__(kThreadsSolve, 1)
fwd_tc_solve_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmO,
                    const __grid_constant__ CUtensorMap tmS, FwdArgs a, long long ntiles) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_bars[2 * B_PER_CHAIN + 1];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    unsigned char *smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    const int tid = threadIdx.x;
    const uint32_t bars = smem_u32(&s_bars[0]);
    const uint32_t abort_addr = smem_u32(&s_abort);

    if (tid == 0) {
        s_abort = 0;
        for (int ch = 0; ch < 2; ++ch)
            for (int i = 0; i < B_PER_CHAIN; ++i) {
                const int count = (i == B_RDY || i == B_RDY_ST || i == B_GF0 || i == B_GF1) ? 16 : 1;
                asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(chain_bar(bars, ch, i)), "r"(count));
            }
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bars + 8 * 2 * B_PER_CHAIN));   // final drain
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
    ChainScalars *const sc0 = reinterpret_cast<ChainScalars *>(smem + OFF_SC);
    auto chain_sc = [&](int ch) { return reinterpret_cast<ChainScalars *>(smem + OFF_SC + ch * (SC_BYTES / 2)); };
    (void)sc0;

    // this block's tiles: a contiguous range, chain ch takes every second one
    const long long t_lo = (ntiles * blockIdx.x) / gridDim.x, t_hi = (ntiles * (blockIdx.x + 1)) / gridDim.x;
    const int n_mine = (int)(t_hi - t_lo);
    auto chain_tiles = [&](int ch) { return (n_mine - ch + 1) / 2; };
    const bool solve_only = EXTRA && a.solve_only != 0;   // the result is the solve itself: no V, no U, no output product
    const float *const beta_p = EXTRA ? a.beta : nullptr;
    const float *const alpha_p = EXTRA ? a.alpha : nullptr;
    const bool mix = alpha_p != nullptr && !solve_only;   // alpha-connection: the read uses alpha x + (1 - alpha) q

    if (tid >= CT) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsHelper));
        const int hw = (tid - CT) >> 5, lane = tid & 31;
        if (hw == 0) {
            // ================= gate scalars of every tile, one tile ahead of the compute warps =================
            const int kmax = max(chain_tiles(0), chain_tiles(1));
            for (int k = 0; k < kmax; ++k) {
                for (int ch = 0; ch < 2; ++ch) {
                    if (k >= chain_tiles(ch)) continue;
                    if (k >= 2) wait_bar(chain_bar(bars, ch, B_GF0 + (k & 1)), (uint32_t)(((k - 2) >> 1) & 1), abort_addr);
                    const TileInfo ti = tile_info(a, t_lo + ch + 2 * k);
                    GateScalars *g = &chain_sc(ch)->g[k & 1];
                    float run = 0.f;
#pragma unroll 1
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
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(chain_bar(bars, ch, B_GS0 + (k & 1)));
                }
            }
        } else if (hw == 1) {
            // ================= TMA: loads of every tile's K, H_0, q; stores of the output tiles =================
            if (lane == 0) {
                auto load_kh = [&](int ch, int k) {      // K goes with H_0 on one barrier
                    const TileInfo ti = tile_info(a, t_lo + ch + 2 * k);
                    const uint32_t cb = sbase + ch * CH_STRIDE;
                    const uint32_t bar = chain_bar(bars, ch, B_LD_KH);
                    mbar_expect_tx(bar, 65536u);
                    tma_load_tile3(&tmK, cb + BUF_K, bar, ti.h * D, ti.n * NT, ti.b);
                    tma_load_tile2(&tmS, cb + BUF_H, bar, (int)((t_lo + ch + 2 * k) * 256));
                };
                auto load_q = [&](int ch, int k) {
                    const TileInfo ti = tile_info(a, t_lo + ch + 2 * k);
                    const uint32_t bar = chain_bar(bars, ch, B_LD_Q);
                    mbar_expect_tx(bar, 32768u);
                    tma_load_tile3(&tmQ, sbase + ch * CH_STRIDE + BUF_D, bar, ti.h * D, ti.n * NT, ti.b);
                };
                // the inputs do not depend on the state kernel; its per-tile states do
                for (int ch = 0; ch < 2; ++ch)
                    if (chain_tiles(ch) > 0) load_q(ch, 0);
                asm volatile("griddepcontrol.wait;" ::: "memory");
                for (int ch = 0; ch < 2; ++ch)
                    if (chain_tiles(ch) > 0) load_kh(ch, 0);
                int k_done[2] = {0, 0};
                uint32_t polls = 0;
                while (k_done[0] < chain_tiles(0) || k_done[1] < chain_tiles(1)) {
                    for (int ch = 0; ch < 2; ++ch) {
                        const int k = k_done[ch];
                        if (k >= chain_tiles(ch)) continue;
                        if (!aborted(abort_addr) && !mbar_test(chain_bar(bars, ch, B_RDY_ST), (uint32_t)(k & 1))) {
                            if (++polls > (1u << 28)) asm volatile("st.volatile.shared.b32 [%0], %1;" ::"r"(abort_addr), "r"(1) : "memory");
                            continue;
                        }
                        polls = 0;
                        const TileInfo ti = tile_info(a, t_lo + ch + 2 * k);
                        const uint32_t cb = sbase + ch * CH_STRIDE;
                        for (int hf = 0; hf < 2; ++hf)     // rows past the sequence are clipped
                            asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];" ::
                                             "l"(reinterpret_cast<uint64_t>(&tmO)), "r"(ti.h * D + 64 * hf), "r"(ti.n * NT),
                                         "r"(ti.b), "r"(cb + BUF_D + 16384 * hf)
                                         : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        const bool more = k + 1 < chain_tiles(ch) && !aborted(abort_addr);
                        if (more) load_kh(ch, k + 1);
                        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the staged tile has been read
                        if (more) load_q(ch, k + 1);
                        k_done[ch] = k + 1;
                    }
                }
                asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // output stores are complete
            }
        } else if (hw == 2) {
            // ================================ MMA issuing thread ================================
            if (lane == 0) {
                const uint32_t base14 = (sbase >> 4) & 0x3FFF;
                const int ops_per_tile = 1 + 2 * a.n_iter + (solve_only ? 0 : 3);
                int done[2] = {0, 0};       // batches issued per chain
                const int total[2] = {chain_tiles(0) * ops_per_tile, chain_tiles(1) * ops_per_tile};
                uint32_t polls = 0;
                while (done[0] < total[0] || done[1] < total[1]) {
#pragma unroll
                    for (int ch = 0; ch < 2; ++ch) {
                        if (done[ch] >= total[ch]) continue;
                        if (!aborted(abort_addr) && !mbar_test(chain_bar(bars, ch, B_RDY), (uint32_t)(done[ch] & 1))) {
                            if (++polls > (1u << 28)) asm volatile("st.volatile.shared.b32 [%0], %1;" ::"r"(abort_addr), "r"(1) : "memory");
                            continue;
                        }
                        polls = 0;
                        fence_after();
                        const int k = done[ch] / ops_per_tile, o = done[ch] - k * ops_per_tile;
                        int op;
                        if (o == 0) op = 0;
                        else if (o <= 2 * a.n_iter) op = 1 + ((o - 1) & 1);
                        else op = 3 + (o - 1 - 2 * a.n_iter);
                        issue_batch(op, base14 + ch * (CH_STRIDE >> 4), tmem + ch * TM_CHAIN, bars, ch, (uint32_t)(k & 1),
                                    abort_addr);
                        ++done[ch];
                    }
                }
                // every product is complete before the block gives its tensor memory back
                mma_commit(bars + 8 * 2 * B_PER_CHAIN);
                if (!mbar_spin_bounded(bars + 8 * 2 * B_PER_CHAIN, 0u))
                    asm volatile("st.volatile.shared.b32 [%0], %1;" ::"r"(abort_addr), "r"(1) : "memory");
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
        cx.sbase = sbase;
        cx.bars = bars;
        cx.tmem = tmem;
        cx.abort_addr = abort_addr;
        const int c = cx.c, cq = cx.cq, l = cx.l;
        const bool adaptive = (a.flags & GKA_FLAG_ADAPTIVE_LAMBDA) != 0;
        // the per-tile states and norms come from the state kernel
        asm volatile("griddepcontrol.wait;" ::: "memory");

        uint64_t xs0[16], xs1[16];          // per chain: -zt_c x_c, this thread's 32 channels as fp32 pairs
        float omega0 = 2.f, omega1 = 2.f;
        int phase[2], iter[2] = {0, 0}, kt[2] = {0, 0};
        uint32_t par = 0;                   // phase bits: bit (4 ch + i) of barrier i in {MMA_S, MMA_R, LD_Q, LD_V}
        phase[0] = chain_tiles(0) > 0 ? PH_SETUP_A : PH_DONE;
        phase[1] = chain_tiles(1) > 0 ? PH_SETUP_A : PH_DONE;
        auto wait_flip = [&](int ch, int which, int bit) {
            wait_bar(chain_bar(bars, ch, which), (par >> (4 * ch + bit)) & 1u, abort_addr);
            par ^= 1u << (4 * ch + bit);
        };

        // ---- pieces that touch a chain's iterate registers: instantiated once per chain
        // x_0: R = q, E_0 = czb q (in place of q), xs = E_0
        auto init_x = [&](uint64_t(&xs)[16], unsigned char *bufd, uint32_t tm_r, float czb) {
#pragma unroll
            for (int g4 = 0; g4 < 4; ++g4) {
                uint4 qv = *reinterpret_cast<const uint4 *>(bufd + tile_off(c, 4 * cq + g4));
                const uint32_t *qq = reinterpret_cast<const uint32_t *>(&qv);
                uint32_t rr[8], pk[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float qa = bf16_lo(qq[u]), qb = bf16_hi(qq[u]);
                    rr[2 * u] = __float_as_uint(qa);
                    rr[2 * u + 1] = __float_as_uint(qb);
                    pk[u] = pack_bf16(czb * qa, czb * qb);
                    xs[4 * g4 + u] = f2_pack(bf16_lo(pk[u]), bf16_hi(pk[u]));
                }
                TMEM_ST8(tm_r + cx.lane_addr + 32 * cq + 8 * g4, rr);
                *reinterpret_cast<uint4 *>(bufd + tile_off(c, 4 * cq + g4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
            tmem_wait_st();
        };
        // one update: e_new = beta e_old + cz (R + lz xs); xs += e_new (as rounded for the operand, unless last)
        auto x_update = [&](uint64_t(&xs)[16], unsigned char *bufd, uint32_t tm_r, float beta, float cz, float lz, bool last) {
            const uint64_t beta2 = f2_pack(beta, beta), cz2 = f2_pack(cz, cz), lz2 = f2_pack(lz, lz);
#pragma unroll
            for (int g4 = 0; g4 < 4; ++g4) {    // 8 channels at a time keeps the transient registers few
                uint32_t r[8];
                TMEM_LD8(tm_r + cx.lane_addr + 32 * cq + 8 * g4, r);
                const uint4 ev = *reinterpret_cast<const uint4 *>(bufd + tile_off(c, 4 * cq + g4));
                const uint32_t *ee = reinterpret_cast<const uint32_t *>(&ev);
                tmem_wait_ld();
                uint32_t pk[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = 4 * g4 + u;
                    const uint64_t res = f2_fma(lz2, xs[i], f2_pack(__uint_as_float(r[2 * u]), __uint_as_float(r[2 * u + 1])));
                    const uint64_t en = f2_fma(cz2, res, f2_mul(beta2, f2_pack(bf16_lo(ee[u]), bf16_hi(ee[u]))));
                    float ea, eb;
                    f2_unpack(en, ea, eb);
                    pk[u] = pack_bf16(ea, eb);
                    xs[i] = f2_add(xs[i], last ? en : f2_pack(bf16_lo(pk[u]), bf16_hi(pk[u])));
                }
                if (!last) *reinterpret_cast<uint4 *>(bufd + tile_off(c, 4 * cq + g4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
        };
        // stage f(-xs) as bf16: hi part (lo == false) or the remainder after the hi part (lo == true), times `scale`
        auto stage_x = [&](const uint64_t(&xs)[16], unsigned char *bufd, bool lo, float scale) {
#pragma unroll
            for (int g4 = 0; g4 < 4; ++g4) {
                uint32_t pk[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float xa, xb;
                    f2_unpack(xs[4 * g4 + u], xa, xb);
                    xa *= -scale;
                    xb *= -scale;
                    uint32_t p = pack_bf16(xa, xb);
                    if (lo) p = pack_bf16(xa - bf16_lo(p), xb - bf16_hi(p));
                    pk[u] = p;
                }
                *reinterpret_cast<uint4 *>(bufd + tile_off(c, 4 * cq + g4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
        };
        // alpha-connection: xs <- alpha xs + (1 - alpha) (-zt q), q re-fetched into `bufq`
        auto mix_x = [&](uint64_t(&xs)[16], const unsigned char *bufq, float alc, float nzt) {
#pragma unroll
            for (int g4 = 0; g4 < 4; ++g4) {
                const uint4 qv = *reinterpret_cast<const uint4 *>(bufq + tile_off(c, 4 * cq + g4));
                const uint32_t *qq = reinterpret_cast<const uint32_t *>(&qv);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float xa, xb;
                    f2_unpack(xs[4 * g4 + u], xa, xb);
                    const float qa = nzt * bf16_lo(qq[u]), qb = nzt * bf16_hi(qq[u]);
                    xs[4 * g4 + u] = f2_pack(fmaf(alc, xa - qa, qa), fmaf(alc, xb - qb, qb));
                }
            }
        };

        // ---- one step of a chain: wait for what the phase needs, do its epilogue, hand the next batch over
        auto step = [&](const int ch) {
            ChainScalars *const cs = chain_sc(ch);
            unsigned char *const cbuf = smem + ch * CH_STRIDE;
            const uint32_t tm_s = tmem + ch * TM_CHAIN + TM_S, tm_r = tmem + ch * TM_CHAIN + TM_R;
            const int k = kt[ch];
            const GateScalars *const gs = &cs->g[k & 1];
            const long long tile = t_lo + ch + 2 * k;
            switch (phase[ch]) {
                case PH_SETUP_A: {
                    // gate scalars (helper warp) and the K, H_0 tiles (TMA) of this tile
                    wait_bar(chain_bar(bars, ch, B_GS0 + (k & 1)), (uint32_t)((k >> 1) & 1), abort_addr);
                    wait_bar(chain_bar(bars, ch, B_LD_KH), (uint32_t)(k & 1), abort_addr);
                    const TileInfo ti = tile_info(a, tile);
                    const bool exact = gs->G2[ti.ntok - 1] < -60.f;  // the tile decays below 2^-60: per-element factors
                    scale_rows(cbuf + BUF_K, gs, exact, tid);
                    fence_async_smem();
                    warp_arrive(chain_bar(bars, ch, B_RDY), l);      // -> FROB
                    phase[ch] = PH_SETUP_B;
                    break;
                }
                case PH_SETUP_B: {
                    const TileInfo ti = tile_info(a, tile);
                    const bool valid = c < ti.ntok;
                    const bool exact = gs->G2[ti.ntok - 1] < -60.f;
                    wait_flip(ch, B_MMA_S, 0);
                    fence_after();
                    // ---- chunk-wise Frobenius norms: per key, k_j^T H_0 k_j and the decayed squared Gram entries of
                    // the earlier keys.  Thread = (key j = c, 32 columns).
                    {
                        float kh = 0.f, gsum = 0.f;
#pragma unroll
                        for (int piece = 0; piece < 2; ++piece) {
                            uint32_t r[16];
                            TMEM_LD16(tm_r + cx.lane_addr + 32 * cq + 16 * piece, r);
                            tmem_wait_ld();
#pragma unroll
                            for (int h2 = 0; h2 < 2; ++h2) {
                                const uint4 kv = *reinterpret_cast<const uint4 *>(cbuf + BUF_K + tile_off(c, 4 * cq + 2 * piece + h2));
                                const uint32_t *pk = reinterpret_cast<const uint32_t *>(&kv);
#pragma unroll
                                for (int u = 0; u < 4; ++u) {
                                    kh = fmaf(__uint_as_float(r[8 * h2 + 2 * u]), bf16_lo(pk[u]), kh);
                                    kh = fmaf(__uint_as_float(r[8 * h2 + 2 * u + 1]), bf16_hi(pk[u]), kh);
                                }
                            }
                        }
                        if (cq <= cx.q) {
                            const float G2j = gs->G2[c];
                            const int lim = (cq == cx.q) ? l : 32;   // keys i < lim come earlier, i == lim is the key itself
                            float gd = 0.f;
#pragma unroll
                            for (int piece = 0; piece < 2; ++piece) {
                                uint32_t r[16];
                                TMEM_LD16(tm_s + cx.lane_addr + 32 * cq + 16 * piece, r);
                                tmem_wait_ld();
#pragma unroll
                                for (int i = 0; i < 16; ++i) {
                                    const int ii = 16 * piece + i;
                                    const float g = __uint_as_float(r[i]);
                                    const float g2 = g * g;
                                    if (ii == lim) gd = g2;
                                    if (!exact) gsum += (ii < lim) ? g2 : 0.f;
                                    else if (ii < lim) gsum = fmaf(ex2_fast(G2j - gs->G2[32 * cq + ii]), g2, gsum);
                                }
                            }
                            gsum = 2.f * gsum + gd;
                        }
                        cs->part[0][cq][c] = kh;
                        cs->part[1][cq][c] = gsum;
                    }
                    fence_before();
                    if (tid == 0) {
                        cs->stop = aborted(abort_addr) ? 1 : 0;
                        cs->exact = exact ? 1 : 0;
                    }
                    asm volatile("bar.sync 1, 512;" ::: "memory");
                    // ---- f_c by an affine scan (s_c = gamma_c^2 s_{c-1} + d_c, s_{-1} = ||H_0||^2), Chebyshev set-up
                    if (tid < NT) {
                        const float hh = a.tile_hh[tile];
                        const float kh = (cs->part[0][0][c] + cs->part[0][1][c]) + (cs->part[0][2][c] + cs->part[0][3][c]);
                        const float gsum = (cs->part[1][0][c] + cs->part[1][1][c]) + (cs->part[1][2][c] + cs->part[1][3][c]);
                        const float G2c = gs->G2[c];
                        // pre-scaled keys: both sums carry 2^(-2 G_c); plain keys: k H_0 k carries zeta_c
                        const float dc = exact ? fmaf(2.f * exp2f(G2c), kh, gsum) : exp2f(2.f * G2c) * fmaf(2.f, kh, gsum);
                        const float s = affine_scan(cx, cs, exp2f(2.f * gs->lg[c]), dc, hh);
                        const float fc = sqrtf(fmaxf(s, 0.f));
                        float lamc = gs->lam[c];
                        if (adaptive) lamc *= fc;
                        const float Lpm = fc + 2.f * lamc;
                        const float rho = fc / Lpm;
                        cs->rho2[c] = rho * rho;
                        cs->czb[c] = valid ? -gs->zt[c] * (2.f / Lpm) : 0.f;
                        cs->lz[c] = lamc * gs->iz[c];
                        if (a.fro_out && valid) a.fro_out[ti.tok0 + (size_t)c * a.heads] = fc;
                    }
                    wait_flip(ch, B_LD_Q, 2);     // q tile has landed
                    asm volatile("bar.sync 1, 512;" ::: "memory");   // the set-up values are published
                    if (cs->stop) {               // the same decision in every thread
                        phase[0] = phase[1] = PH_DONE;
                        break;
                    }
                    {
                        const float czb = cs->czb[c];
                        if (ch == 0) { init_x(xs0, cbuf + BUF_D, tm_r, czb); omega0 = 2.f; }
                        else { init_x(xs1, cbuf + BUF_D, tm_r, czb); omega1 = 2.f; }
                    }
                    iter[ch] = 0;
                    if (a.n_iter > 0) {
                        fence_async_smem();
                        fence_before();
                        warp_arrive(chain_bar(bars, ch, B_RDY), l);   // -> ITER1
                        phase[ch] = PH_P;
                        break;
                    }
                    phase[ch] = PH_X;             // no iteration: x_0 is the final iterate
                }
                // fallthrough (n_iter == 0)
                case PH_X: {
                    const bool have_pass = a.n_iter > 0;
                    const bool last = !have_pass || iter[ch] + 1 == a.n_iter;
                    if (have_pass) {
                        wait_flip(ch, B_MMA_R, 1);
                        fence_after();
                        float &om = ch == 0 ? omega0 : omega1;
                        om = 4.f / (4.f - cs->rho2[c] * om);        // weight schedule of Algorithm 1
                        const float beta = om - 1.f, cz = cs->czb[c] * om, lz = cs->lz[c];
                        if (ch == 0) x_update(xs0, cbuf + BUF_D, tm_r, beta, cz, lz, last);
                        else x_update(xs1, cbuf + BUF_D, tm_r, beta, cz, lz, last);
                    }
                    if (!last) {
                        ++iter[ch];
                        fence_async_smem();
                        fence_before();
                        warp_arrive(chain_bar(bars, ch, B_RDY), l);   // -> ITER1
                        phase[ch] = PH_P;
                        break;
                    }
                    // ---- final iterate
                    if (solve_only) {
                        // the solve is the result: x_c = -xs / zt_c as bf16, stored by TMA
                        const float inv = gs->iz[c];
                        if (ch == 0) stage_x(xs0, cbuf + BUF_D, false, inv);
                        else stage_x(xs1, cbuf + BUF_D, false, inv);
                        fence_async_smem();
                        warp_arrive(chain_bar(bars, ch, B_GF0 + (k & 1)), l);
                        warp_arrive(chain_bar(bars, ch, B_RDY_ST), l);
                        kt[ch] = k + 1;
                        phase[ch] = (k + 1 < chain_tiles(ch)) ? PH_SETUP_A : PH_DONE;
                        break;
                    }
                    if (mix) {
                        // alpha-connection (Section 4.3): the read uses alpha x + (1 - alpha) q; q comes back into the
                        // H_0 buffer, which no product reads any more
                        if (tid == 0) {
                            const TileInfo ti = tile_info(a, tile);
                            const uint32_t bar = chain_bar(bars, ch, B_LD_Q);
                            mbar_expect_tx(bar, 32768u);
                            tma_load_tile3(&tmQ, sbase + ch * CH_STRIDE + BUF_H, bar, ti.h * D, ti.n * NT, ti.b);
                        }
                        wait_flip(ch, B_LD_Q, 2);
                        const float alc = gs->al[c], nzt = cs->czb[c] != 0.f ? -gs->zt[c] : 0.f;   // 0 past the sequence
                        if (ch == 0) mix_x(xs0, cbuf + BUF_H, alc, nzt);
                        else mix_x(xs1, cbuf + BUF_H, alc, nzt);
                        asm volatile("bar.sync 1, 512;" ::: "memory");   // every thread has read q: U_0 may overwrite it
                    }
                    if (tid == 0) {               // U_0 into the H_0 buffer (every product on H_0 is complete)
                        const uint32_t bar = chain_bar(bars, ch, B_LD_U);
                        mbar_expect_tx(bar, 32768u);
                        tma_load_tile2(&tmS, sbase + ch * CH_STRIDE + BUF_H, bar, (int)(tile * 256 + 128));
                    }
                    if (ch == 0) stage_x(xs0, cbuf + BUF_D, false, 1.f);
                    else stage_x(xs1, cbuf + BUF_D, false, 1.f);
                    fence_async_smem();
                    fence_before();
                    warp_arrive(chain_bar(bars, ch, B_RDY), l);       // -> OUT_HI
                    phase[ch] = PH_OUT2;
                    break;
                }
                case PH_P: {
                    wait_flip(ch, B_MMA_S, 0);
                    fence_after();
                    p_epilogue(cx, tm_s, gs->G2, cs->exact != 0, gs->ac[c]);
                    fence_before();
                    warp_arrive(chain_bar(bars, ch, B_RDY), l);       // -> ITER2
                    phase[ch] = PH_X;
                    break;
                }
                case PH_OUT2: {
                    wait_flip(ch, B_MMA_S, 0);                        // the products on X_hi are complete
                    if (ch == 0) stage_x(xs0, cbuf + BUF_D, true, 1.f);
                    else stage_x(xs1, cbuf + BUF_D, true, 1.f);
                    fence_async_smem();
                    warp_arrive(chain_bar(bars, ch, B_RDY), l);       // -> OUT_LO
                    phase[ch] = PH_OUT3;
                    break;
                }
                case PH_OUT3: {
                    const bool exact = cs->exact != 0;
                    wait_flip(ch, B_MMA_S, 0);
                    fence_after();
                    if (tid == 0) {               // the keys are no longer needed: their buffer takes the V tile
                        const TileInfo ti = tile_info(a, tile);
                        const uint32_t bar = chain_bar(bars, ch, B_LD_V);
                        mbar_expect_tx(bar, 32768u);
                        tma_load_tile3(&tmV, sbase + ch * CH_STRIDE + BUF_K, bar, ti.h * D, ti.n * NT, ti.b);
                    }
                    p_epilogue(cx, tm_s, gs->G2, exact, gs->ac[c]);
                    wait_flip(ch, B_LD_V, 3);
                    // Vhat_j = sqrt(beta_j) 2^(-G_j / 2) v_j pairs with the scores on Khat
                    scale_rows(cbuf + BUF_K, gs, exact, tid);
                    fence_async_smem();
                    fence_before();
                    warp_arrive(chain_bar(bars, ch, B_RDY), l);       // -> OUT_PV
                    phase[ch] = PH_OUT4;
                    break;
                }
                case PH_OUT4: {
                    wait_flip(ch, B_MMA_R, 1);
                    fence_after();
                    // O as bf16 into the operand buffer (no product reads it any more), stored by TMA
#pragma unroll
                    for (int piece = 0; piece < 2; ++piece) {
                        uint32_t r[16];
                        TMEM_LD16(tm_r + cx.lane_addr + 32 * cq + 16 * piece, r);
                        tmem_wait_ld();
                        uint32_t pk[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) pk[u] = pack_bf16(__uint_as_float(r[2 * u]), __uint_as_float(r[2 * u + 1]));
                        *reinterpret_cast<uint4 *>(cbuf + BUF_D + tile_off(c, 4 * cq + 2 * piece)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        *reinterpret_cast<uint4 *>(cbuf + BUF_D + tile_off(c, 4 * cq + 2 * piece + 1)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                    }
                    fence_async_smem();
                    fence_before();
                    warp_arrive(chain_bar(bars, ch, B_GF0 + (k & 1)), l);
                    warp_arrive(chain_bar(bars, ch, B_RDY_ST), l);
                    kt[ch] = k + 1;
                    phase[ch] = (k + 1 < chain_tiles(ch)) ? PH_SETUP_A : PH_DONE;
                    break;
                }
                default: break;
            }
        };

        while (phase[0] != PH_DONE || phase[1] != PH_DONE) {
            if (phase[0] != PH_DONE) step(0);
            if (phase[1] != PH_DONE) step(1);
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
    if (a.ev_start) cudaEventRecord(a.ev_start, stream);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)a.plan.G);
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
