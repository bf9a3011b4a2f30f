// tcgen05 path of the chunked GKA forward (bf16 operands, fp32 accumulation) for sm_100a: launcher, the
// segment-summary kernel and the state kernel.  The solve kernel (Algorithm 1 on 128-token tiles) is in
// gka_tc_solve.cu.
//
// The path works on tiles of 128 consecutive tokens of one sequence (two of the paper's chunks: the chunk-wise
// form of Section 4.2.1 is exact for any chunk size).  The state recurrences of eq. (CH),
//     H_t = gamma_t H_{t-1} + beta_t k_t k_t^T,     U_t = gamma_t U_{t-1} + beta_t v_t k_t^T,
// advance tile by tile:  H <- zeta H + K^T (w o K),  U <- zeta U + V^T (w o K)  with zeta the decay of the whole
// tile and w_j the decay from token j to the tile's end (times beta_j).  The state kernel keeps fp32 masters of H
// and U in tensor memory for a whole run of tiles and stores, for every tile, the bf16 operand copies of the
// tile-initial H_0, U_0 and ||H_0||_F^2 (the paper stores the chunk-initial states as well); the solve kernel
// then processes the tiles as independent problems.
//
// Work decomposition (gka_common.cuh): the flat list of tiles is cut into one contiguous range per thread block.
// Where a range ends inside a sequence the summary kernel first computes the decay product and (delta-H,
// delta-U) of its last run, i.e. the run's final state for a zero start state; the state kernel folds the
// summaries of the blocks that hold the earlier part of a sequence into its start state (long chains are
// materialised once by the scan kernel instead).
#include <cuda.h>

#include "gka_common.cuh"
#include "gka_tc_mma.cuh"

namespace gka {
cudaError_t launch_fwd_solve(const FwdArgs &a, cudaStream_t stream);   // gka_tc_solve.cu
namespace {

using namespace tcu;

constexpr int D = 128;
constexpr int NT = kTile;                                // tokens per tile
constexpr int CT = 512;                                  // compute threads; + one warp that issues the products
constexpr int kThreadsState = CT + 32;

// ------------------------------------------------------------------------------------------------------------
// Segment summaries.  The weights are formed in log2 space from the run's total log-decay (one pre-pass over the
// gates) and a running prefix, so every tile is a pure accumulation K^T (w o K), V^T (w o K) into TMEM: no
// rescaling pass.  The kernel streams K and V once: three TMA stages of K and V tiles keep two tiles in flight
// while the third is consumed.  A summarised run never holds the last tile of its sequence, so all its tiles
// are full.
// ------------------------------------------------------------------------------------------------------------
constexpr int SUM_NS = 3;                                // TMA stages
constexpr uint32_t SUM_STAGE = 65536;                    // K tile + V tile
constexpr uint32_t SUM_OFF_KW = SUM_NS * SUM_STAGE;      // w o K
constexpr uint32_t SUM_SMEM = SUM_OFF_KW + 32768 + 1024; // + slack for the 1024-byte alignment of the base
enum { SB_KV0 = 0, SB_MMA = SUM_NS, SB_COUNT };

__global__ void __launch_bounds__(kThreadsState, 1)
fwd_tc_summary_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, FwdArgs a) {
    const WorkPlan &P = a.plan;
    const int item = blockIdx.x;
    // the state kernel may be launched as a programmatic dependent: its blocks may take the SMs that this grid
    // leaves and run their prologue; they wait for this grid's completion before they read a summary
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (!P.cut_out(item)) return;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_bars[SB_COUNT];
    __shared__ uint32_t s_tmem_base;
    __shared__ float s_w[NT], s_ca[4], s_red[16];
    __shared__ int s_req, s_abort;
    unsigned char *smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    const uint32_t sb = smem_u32(smem), bars = smem_u32(&s_bars[0]);
    const int t = threadIdx.x, l = t & 31;

    if (t == 0) {
        s_abort = 0;
        for (int i = 0; i < SB_COUNT; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bars + 8 * i));
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
    const int ntiles = (int)(f1 - f0);
    const uint32_t base14 = (sb >> 4) & 0x3FFF;

    if (t >= CT) {
        // ================================ MMA issuing warp ================================
        for (;;) {
            asm volatile("bar.sync 3, 544;" ::: "memory");         // the compute threads hand over a tile
            const int n = *reinterpret_cast<const volatile int *>(&s_req);
            if (n < 0) break;
            if (l == 0) {
                fence_after();
                const uint32_t kb = base14 + (uint32_t)(n % SUM_NS) * (SUM_STAGE >> 4);
                const uint32_t vb = kb + (32768u >> 4), kwb = base14 + (SUM_OFF_KW >> 4);
                if (n == 0) {
                    mma8_mm<0>(tm_H, kb, kwb, kIdescMM);
                    mma8_mm<0>(tm_U, vb, kwb, kIdescMM);
                } else {
                    mma8_mm<1>(tm_H, kb, kwb, kIdescMM);
                    mma8_mm<1>(tm_U, vb, kwb, kIdescMM);
                }
                mma_commit(bars + 8 * SB_MMA);
            }
            __syncwarp();
        }
    } else {
        // ================================= compute threads =================================
        const int seq = (int)((unsigned)f0 / (unsigned)P.N), b = seq / a.heads, h = seq % a.heads;
        const int n0 = (int)((unsigned)f0 - (unsigned)seq * (unsigned)P.N);   // first tile of the run in its sequence
        const float *grun = a.gate + ((size_t)b * a.T + (size_t)n0 * NT) * a.heads + h;   // token stride: heads
        const float *brun = a.beta ? a.beta + ((size_t)b * a.T + (size_t)n0 * NT) * a.heads + h : nullptr;
        const int ntok_run = ntiles * NT;
        auto issue_tma = [&](int n) {
            const uint32_t dst = sb + (uint32_t)(n % SUM_NS) * SUM_STAGE;
            const uint32_t bar = bars + 8 * (SB_KV0 + n % SUM_NS);
            mbar_expect_tx(bar, 65536u);
            tma_load_tile3(&tmK, dst, bar, h * D, (n0 + n) * NT, b);
            tma_load_tile3(&tmV, dst + 32768, bar, h * D, (n0 + n) * NT, b);
        };
        if (t == 0)
            for (int n = 0; n < ntiles && n < SUM_NS; ++n) issue_tma(n);

        // ---- pre-pass: total log2 decay of the run
        float total = 0.f;
        {
            float s = 0.f;
            for (int i0 = t; i0 < ntok_run; i0 += 4 * CT) {     // four independent loads in flight per thread
                float g[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = i0 + u * CT;
                    g[u] = (i < ntok_run) ? __ldg(grun + (size_t)i * a.heads) : 1.f;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) s += fmaxf(log2f(g[u]), -115.f);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (l == 0) s_red[t >> 5] = s;
            asm volatile("bar.sync 1, 512;" ::: "memory");
#pragma unroll
            for (int i = 0; i < 16; ++i) total += s_red[i];
        }

        // threads 0..127: gate of token t of tile n; fetched one tile ahead, the logarithm is taken when the
        // value is used so that nothing waits for the load
        auto load_gate = [&](int n) -> float {
            const int i = n * NT + t;
            return (t < NT && i < ntok_run) ? __ldg(grun + (size_t)i * a.heads) : 1.f;
        };
        float g_cur = load_gate(0);
        float prefix = 0.f;                    // log2 decay of the tiles before the current one
        for (int n = 0; n < ntiles; ++n) {
            const float g_next = load_gate(n + 1);
            if (t < NT) {
                float incl = fmaxf(log2f(g_cur), -115.f);
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const float up = __shfl_up_sync(0xffffffffu, incl, o);
                    if (l >= o) incl += up;
                }
                if (l == 31) s_ca[t >> 5] = incl;
                asm volatile("bar.sync 2, 128;" ::: "memory");
                float before = 0.f, tile_total = 0.f;
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    if (w < (t >> 5)) before += s_ca[w];
                    tile_total += s_ca[w];
                }
                incl += before;
                // w_j = 2^(decay from token j to the end of the run) = 2^((total - prefix) - incl_j)
                float wt = exp2f((total - prefix) - incl);
                if (brun) wt *= fmaxf(__ldg(brun + (size_t)(n * NT + t) * a.heads), 0.f);   // write strength
                s_w[t] = wt;
                prefix += tile_total;
            }
            // the previous tile's products are done: the w o K buffer and that tile's stage are free
            if (n >= 1) {
                if (!mbar_spin_bounded(bars + 8 * SB_MMA, (uint32_t)((n - 1) & 1))) s_abort = 1;
                if (t == 0 && n + 2 < ntiles) issue_tma(n + 2);
            }
            if (!mbar_spin_bounded(bars + 8 * (SB_KV0 + n % SUM_NS), (uint32_t)((n / SUM_NS) & 1))) s_abort = 1;
            asm volatile("bar.sync 1, 512;" ::: "memory");       // weights are published (and the scan scratch is free)
            const unsigned char *kt = smem + (size_t)(n % SUM_NS) * SUM_STAGE;
            unsigned char *kw = smem + SUM_OFF_KW;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int qi = t + CT * i;                 // 16-byte group index in the 32 KB tile
                const int j = (qi & 1023) >> 3;            // key row of this group
                uint4 v = *reinterpret_cast<const uint4 *>(kt + qi * 16);
                const float wj = s_w[j];
                uint32_t *pv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
                for (int u = 0; u < 4; ++u) pv[u] = pack_bf16(bf16_lo(pv[u]) * wj, bf16_hi(pv[u]) * wj);
                *reinterpret_cast<uint4 *>(kw + qi * 16) = v;
            }
            fence_async_smem();
            if (t == 0) *reinterpret_cast<volatile int *>(&s_req) = n;
            asm volatile("bar.sync 3, 544;" ::: "memory");       // hand the tile to the issuing warp
            g_cur = g_next;
        }
        if (ntiles > 0 && !mbar_spin_bounded(bars + 8 * SB_MMA, (uint32_t)((ntiles - 1) & 1))) s_abort = 1;
        if (t == 0) *reinterpret_cast<volatile int *>(&s_req) = -1;
        asm volatile("bar.sync 3, 544;" ::: "memory");           // releases the issuing warp
        fence_after();
        if (s_abort != 0) {
            if (t == 0 && a.device_status) atomicExch(a.device_status, (int)GKA_ERR_TIMEOUT);
        } else {
            // thread = (row c of dH and of dU, 32 columns)
            const int c = 32 * ((t >> 5) & 3) + l, cq = t >> 7;
            const uint32_t lane_addr = (uint32_t)(32 * ((t >> 5) & 3)) << 16;
            const size_t st = state_floats(D, D);
            float *dst = a.ws.delta + (size_t)item * st + (size_t)c * D + 32 * cq;
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                uint32_t r[32];
                TMEM_LD32(tmem + 128 * which + lane_addr + 32 * cq, r);
                tmem_wait_ld();
                float *p = dst + which * (size_t)D * D;
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    *reinterpret_cast<float4 *>(p + 4 * i) = make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]),
                                                                         __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
            }
            if (t == 0) a.ws.decay[item] = exp2f(total);
        }
    }
    fence_before();
    __syncthreads();
    if (t < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
}

// ------------------------------------------------------------------------------------------------------------
// State kernel.  One block per work item walks its tiles in order.  Thread = (state row c, 32 columns) of both
// masters.  Per tile: the weights w (threads 0..127), w o K into a double-buffered operand tile, then for H and
// for U one pass over the master (bf16 copy of the tile-initial state straight to the workspace, sum of squares
// of H_0, scaling by the tile's decay) followed by the accumulating product of the tile; the product of one
// master runs under the pass over the other.
// ------------------------------------------------------------------------------------------------------------
constexpr uint32_t ST_OFF_K = 0;                 // K tiles, 2 stages
constexpr uint32_t ST_OFF_V = 65536;             // V tiles, 2 stages
constexpr uint32_t ST_OFF_KW = 131072;           // w o K, 2 buffers
constexpr uint32_t ST_SMEM = 196608 + 1024;
enum { TB_K0 = 0, TB_K1, TB_V0, TB_V1, TB_H, TB_U, TB_COUNT };

__device__ __noinline__ void state_seed(uint32_t taddr, const float *state, const float *delta, const float *decay,
                                        int j0, int j1, size_t st, size_t e) {
    // Start of a run: the master's value (this thread's row, 32 columns) is the caller's initial state of the
    // sequence (or zero) carried through the summaries j0 .. j1 - 1: state <- decay_j * state + delta_j.
    float g[32];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float4 v4 = state ? *reinterpret_cast<const float4 *>(state + e + 4 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
        g[4 * i + 0] = v4.x; g[4 * i + 1] = v4.y; g[4 * i + 2] = v4.z; g[4 * i + 3] = v4.w;
    }
    for (int j = j0; j < j1; ++j) {
        // summaries come from the kernel this one may overlap with as its programmatic dependent: ordinary loads
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

// One pass over this thread's part of a master: bf16 copy to `dst` (row-major [128][128], this thread's 32
// columns), optional sum of squares, scaling by the tile's decay.
template <bool SUMSQ>
__device__ __forceinline__ float state_pass(uint32_t taddr, unsigned char *dst, float decay) {
    float ss = 0.f;
#pragma unroll
    for (int piece = 0; piece < 2; ++piece) {
        uint32_t r[16];
        TMEM_LD16(taddr + 16 * piece, r);
        tmem_wait_ld();
        uint32_t pk[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float v0 = __uint_as_float(r[2 * u]), v1 = __uint_as_float(r[2 * u + 1]);
            if (SUMSQ) ss = fmaf(v0, v0, fmaf(v1, v1, ss));
            pk[u] = pack_bf16(v0, v1);
        }
        *reinterpret_cast<uint4 *>(dst + 32 * piece) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        *reinterpret_cast<uint4 *>(dst + 32 * piece + 16) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
#pragma unroll
        for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * decay);
        TMEM_ST16(taddr + 16 * piece, r);
    }
    tmem_wait_st();
    return ss;
}

__global__ void __launch_bounds__(kThreadsState, 1)
fwd_tc_state_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, FwdArgs a) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_bars[TB_COUNT];
    __shared__ uint32_t s_tmem_base;
    __shared__ float s_w[NT], s_ca[4], s_red[16], s_glast;
    __shared__ int s_req, s_abort;
    unsigned char *smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    const uint32_t sb = smem_u32(smem), bars = smem_u32(&s_bars[0]);
    const int t = threadIdx.x, l = t & 31;
    // the solve kernel is launched as a programmatic dependent of this one
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (t == 0) {
        s_abort = 0;
        for (int i = 0; i < TB_COUNT; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bars + 8 * i));
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
    const WorkPlan &P = a.plan;
    const int item = blockIdx.x;
    const long long f_lo = P.lo(item), f_hi = P.lo(item + 1);
    const int n_mine = (int)(f_hi - f_lo);
    const uint32_t base14 = (sb >> 4) & 0x3FFF;

    if (t >= CT) {
        // ================================ MMA issuing warp ================================
        for (;;) {
            asm volatile("bar.sync 3, 544;" ::: "memory");
            const int req = *reinterpret_cast<const volatile int *>(&s_req);
            if (req < 0) break;
            if (l == 0) {
                fence_after();
                const int s = (req >> 1) & 1;                  // stage of the tile
                const uint32_t kwb = base14 + ((ST_OFF_KW + (uint32_t)s * 32768u) >> 4);
                if (req & 1) {                                 // U += V^T (w o K)
                    mma8_mm<1>(tm_U, base14 + ((ST_OFF_V + (uint32_t)s * 32768u) >> 4), kwb, kIdescMM);
                    mma_commit(bars + 8 * TB_U);
                } else {                                       // H += K^T (w o K)
                    mma8_mm<1>(tm_H, base14 + ((ST_OFF_K + (uint32_t)s * 32768u) >> 4), kwb, kIdescMM);
                    mma_commit(bars + 8 * TB_H);
                }
            }
            __syncwarp();
        }
    } else if (n_mine > 0) {
        // ================================= compute threads =================================
        const int q = (t >> 5) & 3, cq = t >> 7, c = 32 * q + l;
        const uint32_t lane_addr = (uint32_t)(32 * q) << 16;
        const size_t st = state_floats(D, D);
        auto wait = [&](int which, uint32_t parity) {     // once a wait has given up the later ones return at once
            if (*reinterpret_cast<volatile int *>(&s_abort) == 0 && !mbar_spin_bounded(bars + 8 * which, parity))
                *reinterpret_cast<volatile int *>(&s_abort) = 1;
        };
        auto post = [&](int req) {
            if (t == 0) *reinterpret_cast<volatile int *>(&s_req) = req;
            asm volatile("bar.sync 3, 544;" ::: "memory");
        };
        // position of tile m of this block
        struct Pos { int seq, n, b, h, ntok; bool run_start, seq_end; size_t tok0; };
        auto pos_of = [&](int m) {
            Pos p;
            const unsigned fu = (unsigned)(f_lo + m);
            p.seq = (int)P.divN.div(fu);
            p.n = (int)(fu - (unsigned)p.seq * (unsigned)P.N);
            p.b = (int)a.divH.div((unsigned)p.seq);
            p.h = p.seq - p.b * a.heads;
            p.ntok = min(NT, a.T - p.n * NT);
            p.run_start = (m == 0) || (p.n == 0);
            p.seq_end = (p.n + 1 == P.N);
            p.tok0 = ((size_t)p.b * a.T + (size_t)p.n * NT) * a.heads + p.h;
            return p;
        };
        auto issue_k = [&](int m) {
            const Pos p = pos_of(m);
            const uint32_t bar = bars + 8 * (TB_K0 + (m & 1));
            mbar_expect_tx(bar, 32768u);
            tma_load_tile3(&tmK, sb + ST_OFF_K + (uint32_t)(m & 1) * 32768u, bar, p.h * D, p.n * NT, p.b);
        };
        auto issue_v = [&](int m) {
            const Pos p = pos_of(m);
            const uint32_t bar = bars + 8 * (TB_V0 + (m & 1));
            mbar_expect_tx(bar, 32768u);
            tma_load_tile3(&tmV, sb + ST_OFF_V + (uint32_t)(m & 1) * 32768u, bar, p.h * D, p.n * NT, p.b);
        };
        if (t == 0) {
            issue_k(0);
            issue_v(0);
            if (n_mine > 1) {
                issue_k(1);
                issue_v(1);
            }
        }
        // first item of the chain of summaries behind this block's start state
        int chain_j0 = item;
        if (P.cut_in(item)) {
            const long long seq_start = (f_lo / P.N) * P.N;
            chain_j0 = item - 1;
            while (P.lo(chain_j0) > seq_start) --chain_j0;
        }
        auto load_scalars = [&](int m, float &g, float &bt) {
            g = 1.f;
            bt = 0.f;
            if (t < NT && m < n_mine) {
                const Pos p = pos_of(m);
                if (t < p.ntok) {
                    g = __ldg(a.gate + p.tok0 + (size_t)t * a.heads);
                    bt = a.beta ? fmaxf(__ldg(a.beta + p.tok0 + (size_t)t * a.heads), 0.f) : 1.f;
                }
            }
        };
        float g_cur, b_cur;
        load_scalars(0, g_cur, b_cur);
        // summaries and start states are read after this point only
        asm volatile("griddepcontrol.wait;" ::: "memory");

        uint32_t n_h = 0, n_u = 0;       // products posted so far (phase counters of the completion barriers)
        for (int m = 0; m < n_mine; ++m) {
            const int s = m & 1;
            const Pos p = pos_of(m);
            float g_next, b_next;
            load_scalars(m + 1, g_next, b_next);
            // ---- weights of the tile's tokens: w_j = beta_j 2^(G_last - G_j), 0 past the sequence
            if (t < NT) {
                float incl = fmaxf(log2f(g_cur), -115.f);
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const float up = __shfl_up_sync(0xffffffffu, incl, o);
                    if (l >= o) incl += up;
                }
                if (l == 31) s_ca[t >> 5] = incl;
                asm volatile("bar.sync 2, 128;" ::: "memory");
                float before = 0.f, tile_total = 0.f;
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    if (w < (t >> 5)) before += s_ca[w];
                    tile_total += s_ca[w];
                }
                incl += before;
                s_w[t] = b_cur * exp2f(tile_total - incl);       // b_cur is 0 past the sequence
                if (t == 0) s_glast = tile_total;
            }
            wait(TB_K0 + s, (uint32_t)((m >> 1) & 1));
            asm volatile("bar.sync 1, 512;" ::: "memory");       // weights are published
            const float decay = exp2f(s_glast);
            // ---- w o K (the buffer was last read by the products of tile m - 2, which are complete: the waits
            // of tile m - 1 below covered them)
            {
                const unsigned char *kt = smem + ST_OFF_K + (size_t)s * 32768;
                unsigned char *kw = smem + ST_OFF_KW + (size_t)s * 32768;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int qi = t + CT * i;
                    const int j = (qi & 1023) >> 3;
                    uint4 v = *reinterpret_cast<const uint4 *>(kt + qi * 16);
                    const float wj = s_w[j];
                    uint32_t *pv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
                    for (int u = 0; u < 4; ++u) pv[u] = pack_bf16(bf16_lo(pv[u]) * wj, bf16_hi(pv[u]) * wj);
                    *reinterpret_cast<uint4 *>(kw + qi * 16) = v;
                }
                fence_async_smem();
            }
            const long long tile = f_lo + m;
            unsigned char *hu = a.tile_hu + (size_t)tile * kTileStateBytes + (size_t)c * 256 + 64 * cq;
            const bool chained = p.run_start && p.n != 0;
            const float *seed_state = (chained && a.start_from_scan) ? a.ws.start + (size_t)item * st
                                      : (a.state_in ? a.state_in + (size_t)p.seq * st : nullptr);
            const int sj0 = (chained && !a.start_from_scan) ? chain_j0 : 0, sj1 = (chained && !a.start_from_scan) ? item : 0;
            // ---- H: the previous tile's product is complete, pass, this tile's product
            if (n_h > 0) wait(TB_H, (n_h - 1) & 1u);
            fence_after();
            if (t == 0 && m >= 1 && m + 1 < n_mine) issue_k(m + 1);     // the K stage of tile m - 1 is free
            if (p.run_start)
                state_seed(tm_H + lane_addr + 32 * cq, seed_state, a.ws.delta, a.ws.decay, sj0, sj1, st, (size_t)c * D + 32 * cq);
            {
                float hs = state_pass<true>(tm_H + lane_addr + 32 * cq, hu, decay);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) hs += __shfl_xor_sync(0xffffffffu, hs, o);
                if (l == 0) s_red[t >> 5] = hs;
            }
            fence_before();
            post(2 * s);
            ++n_h;
            if (t == 0) {
                float hh = 0.f;
#pragma unroll
                for (int i = 0; i < 16; ++i) hh += s_red[i];
                a.tile_hh[tile] = hh;
            }
            // ---- U
            if (n_u > 0) wait(TB_U, (n_u - 1) & 1u);
            fence_after();
            if (t == 0 && m >= 1 && m + 1 < n_mine) issue_v(m + 1);
            if (p.run_start)
                state_seed(tm_U + lane_addr + 32 * cq, seed_state, a.ws.delta, a.ws.decay, sj0, sj1, st,
                           (size_t)D * D + (size_t)c * D + 32 * cq);
            state_pass<false>(tm_U + lane_addr + 32 * cq, hu + 32768, decay);
            wait(TB_V0 + s, (uint32_t)((m >> 1) & 1));
            fence_before();
            post(2 * s + 1);
            ++n_u;
            // ---- final state of the sequence
            if (p.seq_end && a.state_out) {
                wait(TB_H, (n_h - 1) & 1u);
                wait(TB_U, (n_u - 1) & 1u);
                fence_after();
                float *so = a.state_out + (size_t)p.seq * st + (size_t)c * D + 32 * cq;
#pragma unroll
                for (int which = 0; which < 2; ++which) {
                    uint32_t r[32];
                    TMEM_LD32(tmem + 128 * which + lane_addr + 32 * cq, r);
                    tmem_wait_ld();
                    float *pp = so + which * (size_t)D * D;
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        *reinterpret_cast<float4 *>(pp + 4 * i) = make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]),
                                                                              __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
                }
                fence_before();
            }
            g_cur = g_next;
            b_cur = b_next;
        }
        // every product is complete before the block leaves (and gives its tensor memory back)
        if (n_h > 0) wait(TB_H, (n_h - 1) & 1u);
        if (n_u > 0) wait(TB_U, (n_u - 1) & 1u);
        post(-1);
        if (t == 0 && s_abort != 0 && a.device_status) atomicExch(a.device_status, (int)GKA_ERR_TIMEOUT);
    } else {
        if (t == 0) *reinterpret_cast<volatile int *>(&s_req) = -1;
        asm volatile("bar.sync 3, 544;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    if (t < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
}

}  // namespace

bool fwd_tc_available() { return get_encode_fn() != nullptr; }

cudaError_t launch_fwd_tc(const FwdArgs &a_in, cudaStream_t stream) {
    FwdArgs a = a_in;
    cudaError_t err = cudaSuccess;
    bool any_cut = false;
    int longest = 0;                   // most summaries behind any item's start state
    for (int i = 0; i + 1 < a.plan.G; ++i) any_cut |= a.plan.cut_out(i);
    for (int i = 1; i < a.plan.G && any_cut; ++i) {
        if (!a.plan.cut_in(i)) continue;
        const long long seq_start = (a.plan.lo(i) / a.plan.N) * a.plan.N;
        int j0 = i - 1;
        while (a.plan.lo(j0) > seq_start) --j0;
        longest = (i - j0) > longest ? (i - j0) : longest;
    }
    // Short chains are folded by the state kernel's blocks themselves; long ones (a sequence spread over many
    // work items) would make every block re-read its whole chain, so the scan kernel materialises the start
    // states once instead.
    a.start_from_scan = longest > 4 ? 1 : 0;
    alignas(64) CUtensorMap tmK, tmV;      // boxes of 128 tokens x 64 channels
    const int cols = a.heads * D;
    if (!make_tile_map(&tmK, a.k, a.B, a.T, cols, NT) || !make_tile_map(&tmV, a.v, a.B, a.T, cols, NT))
        return cudaErrorInvalidValue;
    if (any_cut) {
        err = cudaFuncSetAttribute(fwd_tc_summary_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SUM_SMEM);
        if (err != cudaSuccess) return err;
        fwd_tc_summary_kernel<<<a.plan.G, kThreadsState, SUM_SMEM, stream>>>(tmK, tmV, a);
        if (a.start_from_scan) {
            err = launch_fwd_scan(a, (int)state_floats(D, D), stream, true);
            if (err != cudaSuccess) return err;
        }
        a.after_summary = 1;
    }
    err = cudaFuncSetAttribute(fwd_tc_state_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ST_SMEM);
    if (err != cudaSuccess) return err;
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)a.plan.G);
        cfg.blockDim = dim3(kThreadsState);
        cfg.dynamicSmemBytes = ST_SMEM;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = a.after_summary ? 1 : 0;
        err = cudaLaunchKernelEx(&cfg, fwd_tc_state_kernel, tmK, tmV, a);
        if (err != cudaSuccess) return err;
    }
    return launch_fwd_solve(a, stream);
}

}  // namespace gka
