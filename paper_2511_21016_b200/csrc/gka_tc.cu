// tcgen05 / TMEM chunk-wise GKA forward (bf16 operands, fp32 accumulation) for sm_100a.
//
// One persistent thread block per SM walks its range of chunks (gka_common.cuh explains the work
// decomposition).  The block has NSLOT "slots"; a slot is one warpgroup of 128 threads that owns one
// chunk of C = 64 tokens at a time, so with NSLOT = 2 the tensor pipe works on one chunk while the
// CUDA cores run the element-wise part of the other.  Slots take chunks alternately.
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

#include "gka_common.cuh"

namespace gka {
namespace {

constexpr int D = 128;
constexpr int C = kChunk;
constexpr int WG = 128;

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
    float dj[C];        // Frobenius increments
    float4 coef[2][C];  // per-iteration (sigma, beta, A, zt)
    float red[8];
    float hh;           // ||H_0||_F^2
    int clamped;        // chunk decays below 2^-60 somewhere
};
constexpr uint32_t SLOT_BYTES = OFF_SC + 4096;
static_assert(sizeof(SlotScalars) <= 4096, "scalar block too large");

// ---- TMEM columns
constexpr uint32_t TM_H = 0, TM_U = 128, TM_Y0 = 256, TM_SPARE = 320, TM_Y1 = 384, TM_S = 448;

enum { BAR_TMA = 0, BAR_A, BAR_B, BAR_COUNT };   // per-slot mbarriers

__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes,
                                              uint32_t layout_type) {
    return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) | ((uint64_t)1 << 46) |
           ((uint64_t)(layout_type & 7) << 61);
}
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, int a_mn, int b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem), "l"(da), "l"(db),
                 "r"(idesc), "r"(acc)
                 : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void wg_sync(int slot) { asm volatile("bar.sync %0, 128;" ::"r"(slot + 1) : "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

#define TMEM_LD16(taddr, r)                                                                                   \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];" \
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),       \
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])  \
                 : "r"(taddr)                                                                                             \
                 : "memory")
#define TMEM_LD32(taddr, r)                                                                                   \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"         \
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"                              \
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),       \
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), \
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]),            \
                   "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]),            \
                   "=r"(r[30]), "=r"(r[31])                                                                               \
                 : "r"(taddr)                                                                                             \
                 : "memory")
#define TMEM_ST32(taddr, r)                                                                                   \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"  \
                 "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),                        \
                 "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),      \
                 "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]),          \
                 "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]),         \
                 "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])                      \
                 : "memory")

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&p);
}
__device__ __forceinline__ float bf16_lo(uint32_t p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t p) { return __uint_as_float(p & 0xFFFF0000u); }
__device__ __forceinline__ float ex2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct TcParams {
    FwdArgs a;
};

// Everything one warpgroup needs to know about itself.
struct SlotCtx {
    int slot, t, warp_q;          // slot index, thread in warpgroup (= TMEM lane), warp within warpgroup
    uint32_t sbase;               // shared address of the slot's buffers
    unsigned char *sptr;          // generic pointer to the same
    SlotScalars *sc;
    uint32_t bars;                // shared address of the slot's mbarriers
    uint32_t tmem;                // TMEM base
    uint32_t tm_y, tm_s, tm_kh;   // accumulator addresses (lane offset included for tm_s)
    uint32_t lane_addr;           // (32 * warp_q) << 16
    uint32_t ph[BAR_COUNT];       // phase parity of each mbarrier
    volatile int *abort_flag;
    int *device_status;
};

__device__ __forceinline__ void slot_wait(SlotCtx &cx, int which) {
    if (*cx.abort_flag == 0) {
        if (!mbar_wait_bounded(cx.bars + 8 * which, cx.ph[which])) {
            *cx.abort_flag = 1;
            if (cx.device_status) atomicExch(cx.device_status, (int)GKA_ERR_TIMEOUT);
        }
    }
    cx.ph[which] ^= 1u;
}

// Masked score epilogue: S^T (TMEM, M = 64 layout) -> P operand in shared memory.
__device__ __forceinline__ void p_epilogue(SlotCtx &cx) {
    const int l = cx.t & 31;
    const bool valid = (l >> 4) == cx.slot;
    const int j = 16 * cx.warp_q + (l & 15);
    const SlotScalars *sc = cx.sc;
    const float bj = -sc->G2[j];
    const float invz = exp2f(fminf(bj, 126.f));
    const bool clamped = sc->clamped != 0;
    unsigned char *prow = cx.sptr + OFF_P + j * 128;
#pragma unroll
    for (int piece = 0; piece < 2; ++piece) {
        uint32_t r[32];
        TMEM_LD32(cx.tm_s + cx.lane_addr + 32 * piece, r);
        tmem_wait_ld();
        if (valid) {
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                uint32_t pk[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int c0 = 32 * piece + 8 * ch + 2 * u;
                    float f0, f1;
                    if (!clamped) {
                        f0 = invz; f1 = invz;
                    } else {
                        f0 = ex2_fast(sc->ac[c0] + bj);
                        f1 = ex2_fast(sc->ac[c0 + 1] + bj);
                    }
                    const float p0 = (j <= c0) ? __uint_as_float(r[8 * ch + 2 * u]) * f0 : 0.f;
                    const float p1 = (j <= c0 + 1) ? __uint_as_float(r[8 * ch + 2 * u + 1]) * f1 : 0.f;
                    pk[u] = pack_bf16(p0, p1);
                }
                const int chunk = (4 * piece + ch) ^ (j & 7);
                *reinterpret_cast<uint4 *>(prow + chunk * 16) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
        }
    }
}

template <int NSLOT>
__global__ void __launch_bounds__(WG *NSLOT, 1)
fwd_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, FwdArgs a) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_bars[NSLOT * BAR_COUNT + 2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    unsigned char *smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    const int tid = threadIdx.x;
    const int slot = tid / WG;
    SlotCtx cx;
    cx.slot = slot;
    cx.t = tid % WG;
    cx.warp_q = cx.t >> 5;
    cx.sptr = smem + (size_t)slot * SLOT_BYTES;
    cx.sbase = smem_u32(cx.sptr);
    cx.sc = reinterpret_cast<SlotScalars *>(cx.sptr + OFF_SC);
    cx.bars = smem_u32(&s_bars[slot * BAR_COUNT]);
    cx.lane_addr = (uint32_t)(32 * cx.warp_q) << 16;
#pragma unroll
    for (int i = 0; i < BAR_COUNT; ++i) cx.ph[i] = 0;
    cx.abort_flag = &s_abort;
    cx.device_status = a.device_status;
    const uint32_t tokH = smem_u32(&s_bars[NSLOT * BAR_COUNT]);
    const uint32_t tokU = tokH + 8;
    SlotScalars *sc = cx.sc;
    const int t = cx.t;

    if (tid == 0) {
        s_abort = 0;
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
    cx.tmem = s_tmem_base;
    cx.tm_y = cx.tmem + (slot == 0 ? TM_Y0 : TM_Y1);
    cx.tm_kh = cx.tmem + (slot == 0 ? TM_Y0 : TM_SPARE) + ((uint32_t)(16 * slot) << 16);
    cx.tm_s = cx.tmem + TM_S + ((uint32_t)(16 * slot) << 16);
    const uint32_t tm_H = cx.tmem + TM_H, tm_U = cx.tmem + TM_U;

    // ---- descriptors (k-step 0); later k-steps add a constant to the low word
    const uint64_t dK_k = make_desc(cx.sbase + OFF_K, 16, 1024, 2);      // K as K-major (rows = keys)
    const uint64_t dK_mn = make_desc(cx.sbase + OFF_K, 8192, 1024, 2);   // K as MN-major (rows = channels)
    const uint64_t dV_mn = make_desc(cx.sbase + OFF_V, 8192, 1024, 2);
    const uint64_t dKw_mn = make_desc(cx.sbase + OFF_KW, 8192, 1024, 2);
    const uint64_t dH_k = make_desc(cx.sbase + OFF_H, 16, 1024, 2);      // H_0 / U_0, K-major
    const uint64_t dX_mn = make_desc(cx.sbase + OFF_X, 8192, 1024, 2);
    const uint64_t dP_mn = make_desc(cx.sbase + OFF_P, 8192, 1024, 2);
    constexpr uint32_t I_S = make_idesc(64, 64, 0, 1);
    constexpr uint32_t I_Y1 = make_idesc(128, 64, 0, 1);
    constexpr uint32_t I_Y2 = make_idesc(128, 64, 1, 1);
    constexpr uint32_t I_ADV = make_idesc(128, 128, 1, 1);
    constexpr uint32_t I_KH = make_idesc(64, 128, 0, 0);
    constexpr uint32_t I_GR = make_idesc(64, 64, 0, 0);
    // K-major operand with two 64-column boxes: k-step ks -> box ks/4 (stride `box` bytes), +32 B per step inside
    auto kmaj_step = [](uint64_t d0, int ks, uint32_t box_bytes) {
        return d0 + (uint64_t)(((ks >> 2) * box_bytes + (ks & 3) * 32) >> 4);
    };
    auto mn_step = [](uint64_t d0, int ks) { return d0 + (uint64_t)((ks * 2048) >> 4); };

    const WorkPlan &P = a.plan;
    const int item = blockIdx.x;
    const long long f_lo = P.lo(item), f_hi = P.lo(item + 1);
    const __nv_bfloat16 *gq = reinterpret_cast<const __nv_bfloat16 *>(a.q);
    __nv_bfloat16 *gout = reinterpret_cast<__nv_bfloat16 *>(a.out);
    const size_t st = state_floats(D, D);
    const bool adaptive = (a.flags & GKA_FLAG_ADAPTIVE_LAMBDA) != 0;

    auto issue_tma = [&](long long f) {   // thread 0 of the warpgroup: K and V tiles of flat chunk f
        const int seq = (int)(f / P.N), n = (int)(f % P.N);
        const int b = seq / a.heads, h = seq % a.heads;
        const int y = b * a.T + n * C;
        const uint32_t bar = cx.bars + 8 * BAR_TMA;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(32768u) : "memory");
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int x = h * D + 64 * half;
            asm volatile(
                "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::
                    "r"(cx.sbase + OFF_K + 8192 * half), "l"(reinterpret_cast<uint64_t>(&tmK)), "r"(x), "r"(y), "r"(bar)
                : "memory");
            asm volatile(
                "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::
                    "r"(cx.sbase + OFF_V + 8192 * half), "l"(reinterpret_cast<uint64_t>(&tmV)), "r"(x), "r"(y), "r"(bar)
                : "memory");
        }
    };

    // first chunk of this slot
    if (t == 0 && f_lo + slot < f_hi) issue_tma(f_lo + slot);

    for (long long f = f_lo + slot; f < f_hi; f += NSLOT) {
        const long long m = f - f_lo;              // index of this chunk inside the block's range
        const int seq = (int)(f / P.N), n = (int)(f % P.N);
        const int b = seq / a.heads, h = seq % a.heads;
        const size_t tok0 = ((size_t)b * a.T + (size_t)n * C) * a.heads + h;
        const bool run_start = (m == 0) || (n == 0);
        const bool seq_end = (n == P.N - 1);
        const float *init_src = nullptr;           // where a run's start state comes from (nullptr = zero)
        if (run_start) init_src = (n == 0) ? (a.state_in ? a.state_in + (size_t)seq * st : nullptr)
                                           : a.ws.start + (size_t)item * st;

        // ---- q for this thread's channel, all 64 tokens, packed bf16 pairs (issued early)
        uint32_t qp[32];
        {
            const unsigned short *qs = reinterpret_cast<const unsigned short *>(gq) + tok0 * D + t;
            const size_t rs = (size_t)a.heads * D;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const uint32_t lo = qs[(size_t)(2 * i) * rs], hi = qs[(size_t)(2 * i + 1) * rs];
                qp[i] = lo | (hi << 16);
            }
        }

        // ---- gates (threads 0..63 own token c = t for scalar bookkeeping)
        if (t < C) {
            const float g = a.gate[tok0 + (size_t)t * a.heads];
            sc->w[t] = fmaxf(log2f(g), -115.f);     // temporary: log2 gamma
            sc->lam[t] = a.lam[tok0 + (size_t)t * a.heads];
        }
        wg_sync(slot);
        float G2c = 0.f;
        if (t < C) {
            for (int i = 0; i <= t; ++i) G2c += sc->w[i];
        }
        wg_sync(slot);
        if (t < C) {
            sc->G2[t] = G2c;
            const float mc = fmaxf(G2c, -60.f);
            sc->zt[t] = exp2f(mc);
            sc->ac[t] = G2c - mc;
            if (t == C - 1) sc->clamped = (G2c < -60.f) ? 1 : 0;
        }
        wg_sync(slot);
        if (t < C) sc->w[t] = exp2f(sc->G2[C - 1] - sc->G2[t]);
        const float zetaC = exp2f(sc->G2[C - 1]);

        // ---- K, V tiles have landed
        slot_wait(cx, BAR_TMA);

        // ---- w o K (same swizzled positions as K)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int qi = t + WG * i;                 // 16-byte chunk index in the 16 KB tile
            const int j = (qi & 511) >> 3;             // key row of this chunk
            uint4 v = *reinterpret_cast<const uint4 *>(cx.sptr + OFF_K + qi * 16);
            const float wj = sc->w[j];
            uint32_t *pv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
            for (int u = 0; u < 4; ++u) pv[u] = pack_bf16(bf16_lo(pv[u]) * wj, bf16_hi(pv[u]) * wj);
            *reinterpret_cast<uint4 *>(cx.sptr + OFF_KW + qi * 16) = v;
        }

        // ---- H master: wait for the previous chunk's advance, then one pass: ||H_0||^2, bf16 copy, scale
        if (NSLOT == 2 && m > 0) {   // chunk m - 1 (the other slot's) has finished its H work
            if (*cx.abort_flag == 0 && !mbar_wait_bounded(tokH, (uint32_t)((m - 1) & 1))) *cx.abort_flag = 1;
        }
        fence_after();
        {
            float hh = 0.f;
            const float *src = (run_start && init_src) ? init_src + (size_t)t * D : nullptr;
#pragma unroll
            for (int piece = 0; piece < 4; ++piece) {
                uint32_t r[32];
                if (!run_start) {
                    TMEM_LD32(tm_H + cx.lane_addr + 32 * piece, r);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        float4 v4 = src ? *reinterpret_cast<const float4 *>(src + 32 * piece + 4 * i)
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
                        r[4 * i + 0] = __float_as_uint(v4.x); r[4 * i + 1] = __float_as_uint(v4.y);
                        r[4 * i + 2] = __float_as_uint(v4.z); r[4 * i + 3] = __float_as_uint(v4.w);
                    }
                }
                unsigned char *hrow = cx.sptr + OFF_H + (piece >> 1) * 16384 + t * 128;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t pk[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float v0 = __uint_as_float(r[8 * ch + 2 * u]), v1 = __uint_as_float(r[8 * ch + 2 * u + 1]);
                        hh = fmaf(v0, v0, fmaf(v1, v1, hh));
                        pk[u] = pack_bf16(v0, v1);
                    }
                    const int chunk = (4 * (piece & 1) + ch) ^ (t & 7);
                    *reinterpret_cast<uint4 *>(hrow + chunk * 16) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * zetaC);
                TMEM_ST32(tm_H + cx.lane_addr + 32 * piece, r);
            }
            tmem_wait_st();
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) hh += __shfl_xor_sync(0xffffffffu, hh, o);
            if ((t & 31) == 0) sc->red[cx.warp_q] = hh;
        }
        fence_async_smem();
        fence_before();
        wg_sync(slot);
        if (t == 0) {
            fence_after();
            // H advance: Hm += K^T (w o K);  K H_0 (M = 64 keys, N = 128);  Gram K K^T
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) mma_ss(tm_H, mn_step(dK_mn, ks), mn_step(dKw_mn, ks), I_ADV, 1);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                mma_ss(cx.tm_kh, kmaj_step(dK_k, ks, 8192), kmaj_step(dH_k, ks, 16384), I_KH, ks > 0);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                mma_ss(cx.tm_s, kmaj_step(dK_k, ks, 8192), kmaj_step(dK_k, ks, 8192), I_GR, ks > 0);
            mma_commit(cx.bars + 8 * BAR_A);
        }
        if (t == 0) sc->hh = sc->red[0] + sc->red[1] + sc->red[2] + sc->red[3];
        slot_wait(cx, BAR_A);
        fence_after();

        // ---- chunk-wise Frobenius norms: d_j, then f_c
        {
            const int l = t & 31;
            const bool valid = (l >> 4) == slot;
            const int j = 16 * cx.warp_q + (l & 15);
            float aj = 0.f;
#pragma unroll
            for (int piece = 0; piece < 4; ++piece) {
                uint32_t r[32];
                TMEM_LD32(cx.tm_kh + cx.lane_addr + 32 * piece, r);
                tmem_wait_ld();
                const unsigned char *krow = cx.sptr + OFF_K + (piece >> 1) * 8192 + j * 128;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    const int chunk = (4 * (piece & 1) + ch) ^ (j & 7);
                    const uint4 kv = *reinterpret_cast<const uint4 *>(krow + chunk * 16);
                    const uint32_t *pk = reinterpret_cast<const uint32_t *>(&kv);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        aj = fmaf(__uint_as_float(r[8 * ch + 2 * u]), bf16_lo(pk[u]), aj);
                        aj = fmaf(__uint_as_float(r[8 * ch + 2 * u + 1]), bf16_hi(pk[u]), aj);
                    }
                }
            }
            float bjs = 0.f;
            const float G2j = sc->G2[j];
#pragma unroll
            for (int piece = 0; piece < 2; ++piece) {
                uint32_t r[32];
                TMEM_LD32(cx.tm_s + cx.lane_addr + 32 * piece, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int ii = 32 * piece + i;
                    const float g = __uint_as_float(r[i]);
                    const float g2 = g * g;
                    if (ii < j) bjs = fmaf(2.f * ex2_fast(G2j - sc->G2[ii]), g2, bjs);
                    else if (ii == j) bjs += g2;
                }
            }
            if (valid) sc->dj[j] = fmaf(2.f * exp2f(G2j) , aj, bjs);
        }
        fence_before();
        wg_sync(slot);
        // H master is final for this chunk, the Frobenius temporaries are consumed
        if (seq_end && a.state_out) {
            fence_after();
            float *dst = a.state_out + (size_t)seq * st + (size_t)t * D;
#pragma unroll
            for (int piece = 0; piece < 4; ++piece) {
                uint32_t r[32];
                TMEM_LD32(tm_H + cx.lane_addr + 32 * piece, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    *reinterpret_cast<float4 *>(dst + 32 * piece + 4 * i) =
                        make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]),
                                    __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
            }
            fence_before();
            wg_sync(slot);
        }
        if (NSLOT == 2 && t == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(tokH) : "memory");

        // ---- f_c, Chebyshev initialisation (threads 0..63: token c = t)
        float omega = 2.f, rho2 = 0.f, s0c = 0.f, lamc = 0.f;
        if (t < C) {
            const float G2t = sc->G2[t];
            float s = exp2f(2.f * G2t) * sc->hh;
            for (int j = 0; j <= t; ++j) s = fmaf(ex2_fast(2.f * (G2t - sc->G2[j])), sc->dj[j], s);
            const float fc = sqrtf(fmaxf(s, 0.f));
            lamc = sc->lam[t];
            if (adaptive) lamc *= fc;
            const float Lpm = fc + 2.f * lamc;
            const float rho = fc / Lpm;
            rho2 = rho * rho;
            s0c = 2.f / Lpm;
            sc->s0[t] = s0c;
            if (a.fro_out) a.fro_out[tok0 + (size_t)t * a.heads] = fc;
        }
        wg_sync(slot);

        // ---- x_0 = 2 q / (L + mu), X' operand
        float xm[C], xp[C];
        {
            unsigned char *xrow = cx.sptr + OFF_X + t * 128;
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
                uint32_t pk[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int c0 = 8 * ch + 2 * u;
                    const float x0 = sc->s0[c0] * bf16_lo(qp[c0 >> 1]);
                    const float x1 = sc->s0[c0 + 1] * bf16_hi(qp[c0 >> 1]);
                    xm[c0] = x0; xm[c0 + 1] = x1;
                    xp[c0] = 0.f; xp[c0 + 1] = 0.f;
                    pk[u] = pack_bf16(x0 * sc->zt[c0], x1 * sc->zt[c0 + 1]);
                }
                *reinterpret_cast<uint4 *>(xrow + ((ch ^ (t & 7)) * 16)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
        }
        fence_async_smem();
        fence_before();
        wg_sync(slot);

        // ---- Algorithm 1: n_iter iterations on the whole chunk (+ one extra score pass for the output)
        for (int it = 0; it <= a.n_iter; ++it) {
            const bool last = (it == a.n_iter);
            if (t == 0) {
                fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    mma_ss(cx.tm_s, kmaj_step(dK_k, ks, 8192), mn_step(dX_mn, ks), I_S, ks > 0);
                mma_commit(cx.bars + 8 * BAR_A);
                if (!last) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        mma_ss(cx.tm_y, kmaj_step(dH_k, ks, 16384), mn_step(dX_mn, ks), I_Y1, ks > 0);
                }
            }
            if (!last && t < C) {   // weight schedule and per-token coefficients of this iteration
                omega = 4.f / (4.f - rho2 * omega);
                const float sigma = s0c * omega, beta = omega - 1.f;
                sc->coef[it & 1][t] = make_float4(sigma, beta, 1.f + beta - sigma * lamc, sc->zt[t]);
            }
            slot_wait(cx, BAR_A);
            fence_after();
            p_epilogue(cx);
            fence_async_smem();
            fence_before();
            wg_sync(slot);
            if (last) break;
            if (t == 0) {
                fence_after();
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) mma_ss(cx.tm_y, mn_step(dK_mn, ks), mn_step(dP_mn, ks), I_Y2, 1);
                mma_commit(cx.bars + 8 * BAR_B);
            }
            slot_wait(cx, BAR_B);
            fence_after();
            {
                const float4 *coef = sc->coef[it & 1];
                unsigned char *xrow = cx.sptr + OFF_X + t * 128;
#pragma unroll
                for (int piece = 0; piece < 4; ++piece) {
                    uint32_t r[16];
                    TMEM_LD16(cx.tm_y + cx.lane_addr + 16 * piece, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int ch = 0; ch < 2; ++ch) {
                        uint32_t pk[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            float xo[2];
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                const int c = 16 * piece + 8 * ch + 2 * u + e;
                                const float4 cf = coef[c];
                                const float qv = e == 0 ? bf16_lo(qp[c >> 1]) : bf16_hi(qp[c >> 1]);
                                const float acc = __uint_as_float(r[8 * ch + 2 * u + e]);
                                const float xn = fmaf(cf.x, qv - acc, fmaf(cf.z, xm[c], -cf.y * xp[c]));
                                xp[c] = xm[c];
                                xm[c] = xn;
                                xo[e] = xn * cf.w;
                            }
                            pk[u] = pack_bf16(xo[0], xo[1]);
                        }
                        const int chunk = (2 * piece + ch) ^ (t & 7);
                        *reinterpret_cast<uint4 *>(xrow + chunk * 16) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
            }
            fence_async_smem();
            fence_before();
            wg_sync(slot);
        }

        // ---- output: U master pass (bf16 copy into the H buffer, scale), O^T = U_0 X'^T + V^T P^T, U advance
        if (NSLOT == 2 && m > 0) {   // chunk m - 1 has written its output and advanced U
            if (*cx.abort_flag == 0 && !mbar_wait_bounded(tokU, (uint32_t)((m - 1) & 1))) *cx.abort_flag = 1;
        }
        fence_after();
        {
            const float *src = (run_start && init_src) ? init_src + (size_t)D * D + (size_t)t * D : nullptr;
#pragma unroll
            for (int piece = 0; piece < 4; ++piece) {
                uint32_t r[32];
                if (!run_start) {
                    TMEM_LD32(tm_U + cx.lane_addr + 32 * piece, r);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        float4 v4 = src ? *reinterpret_cast<const float4 *>(src + 32 * piece + 4 * i)
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
                        r[4 * i + 0] = __float_as_uint(v4.x); r[4 * i + 1] = __float_as_uint(v4.y);
                        r[4 * i + 2] = __float_as_uint(v4.z); r[4 * i + 3] = __float_as_uint(v4.w);
                    }
                }
                unsigned char *hrow = cx.sptr + OFF_H + (piece >> 1) * 16384 + t * 128;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t pk[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        pk[u] = pack_bf16(__uint_as_float(r[8 * ch + 2 * u]), __uint_as_float(r[8 * ch + 2 * u + 1]));
                    const int chunk = (4 * (piece & 1) + ch) ^ (t & 7);
                    *reinterpret_cast<uint4 *>(hrow + chunk * 16) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * zetaC);
                TMEM_ST32(tm_U + cx.lane_addr + 32 * piece, r);
            }
            tmem_wait_st();
        }
        fence_async_smem();
        fence_before();
        wg_sync(slot);
        if (t == 0) {
            fence_after();
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                mma_ss(cx.tm_y, kmaj_step(dH_k, ks, 16384), mn_step(dX_mn, ks), I_Y1, ks > 0);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) mma_ss(cx.tm_y, mn_step(dV_mn, ks), mn_step(dP_mn, ks), I_Y2, 1);
            mma_commit(cx.bars + 8 * BAR_A);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) mma_ss(tm_U, mn_step(dV_mn, ks), mn_step(dKw_mn, ks), I_ADV, 1);
            mma_commit(cx.bars + 8 * BAR_B);
        }
        slot_wait(cx, BAR_A);
        fence_after();
        {
            unsigned short *orow = reinterpret_cast<unsigned short *>(gout) + tok0 * D + t;
            const size_t rs = (size_t)a.heads * D;
#pragma unroll
            for (int piece = 0; piece < 4; ++piece) {
                uint32_t r[16];
                TMEM_LD16(cx.tm_y + cx.lane_addr + 16 * piece, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const __nv_bfloat16 ob = __float2bfloat16_rn(__uint_as_float(r[i]));
                    orow[(size_t)(16 * piece + i) * rs] = *reinterpret_cast<const unsigned short *>(&ob);
                }
            }
        }
        slot_wait(cx, BAR_B);     // U advance done: every tensor-core read of this chunk's tiles is done
        fence_after();
        if (seq_end && a.state_out) {
            float *dst = a.state_out + (size_t)seq * st + (size_t)D * D + (size_t)t * D;
#pragma unroll
            for (int piece = 0; piece < 4; ++piece) {
                uint32_t r[32];
                TMEM_LD32(tm_U + cx.lane_addr + 32 * piece, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    *reinterpret_cast<float4 *>(dst + 32 * piece + 4 * i) =
                        make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]),
                                    __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
            }
        }
        fence_before();
        wg_sync(slot);
        if (t == 0) {
            if (NSLOT == 2) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(tokU) : "memory");
            if (f + NSLOT < f_hi && *cx.abort_flag == 0) issue_tma(f + NSLOT);
        }
        if (*cx.abort_flag != 0) break;
    }

    fence_before();
    __syncthreads();
    if (tid < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(cx.tmem) : "memory");
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D map over a [B*T rows][heads*D columns] bf16 tensor, box = 64 columns x 64 rows, 128-byte swizzle.
bool make_tile_map(CUtensorMap *map, const void *base, int rows, int cols) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, 64};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kSlots = 1;

}  // namespace

bool fwd_tc_available() { return get_encode_fn() != nullptr; }

cudaError_t launch_fwd_tc(const FwdArgs &a, cudaStream_t stream) {
    alignas(64) CUtensorMap tmK, tmV;
    const int rows = a.B * a.T, cols = a.heads * D;
    if (!make_tile_map(&tmK, a.k, rows, cols) || !make_tile_map(&tmV, a.v, rows, cols))
        return cudaErrorInvalidValue;
    cudaError_t err = launch_fwd_summary_scan_bf16_d128(a, stream);
    if (err != cudaSuccess) return err;
    const size_t smem = (size_t)kSlots * SLOT_BYTES + 1024;
    err = cudaFuncSetAttribute(fwd_tc_kernel<kSlots>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    if (a.ev_start) cudaEventRecord(a.ev_start, stream);
    fwd_tc_kernel<kSlots><<<a.plan.G, WG * kSlots, smem, stream>>>(tmK, tmV, a);
    if (a.ev_stop) cudaEventRecord(a.ev_stop, stream);
    return cudaGetLastError();
}

}  // namespace gka
