// tcgen05 path of the chunked GKA forward (bf16 operands, fp32 accumulation) for sm_100a: launcher, the
// segment-summary kernel and the state kernel.  The solve kernel (Algorithm 1 on 128-token tiles) is in
// gka_tc_solve.cu.
//
// The path works on tiles of 128 consecutive tokens of one sequence (two of the paper's chunks: the chunk-wise
// form of Section 4.2.1 is exact for any chunk size).  The state recurrences of eq. (CH),
//     H_t = gamma_t H_{t-1} + beta_t k_t k_t^T,     U_t = gamma_t U_{t-1} + beta_t v_t k_t^T,
// advance tile by tile:  H <- zeta H + K^T diag(w) K,  U <- zeta U + V^T diag(w) K  with zeta the decay of the whole
// tile and w_j the decay from token j to the tile's end (times beta_j).  The state kernel keeps fp32 masters of H
// and U on chip for a whole run of tiles and stores, for every tile, the bf16 operand copies of the
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
constexpr int kThreadsStateK = CT + 64;                  // state kernel: one more warp for the TMA loads and stores

// ------------------------------------------------------------------------------------------------------------
// Both kernels advance a state by whole tiles with the products K~^T K~ and V~^T K~ on rows scaled in place,
// K~_j = sqrt(w_j) k_j and V~_j = sqrt(w_j) v_j (w_j includes the write strength beta_j), so that no weighted copy of
// the keys is needed and three TMA stages of K and V tiles fit: the loads run two tiles ahead.
// ------------------------------------------------------------------------------------------------------------
constexpr int NS = 3;                                    // TMA stages
constexpr uint32_t STAGE = 65536;                        // K tile + V tile
constexpr uint32_t KV_SMEM = NS * STAGE + 1024;          // + slack for the 1024-byte alignment of the base
constexpr uint32_t ST_SMEM = KV_SMEM;

// rows of the K and V tiles of a stage times f[j]
__device__ __forceinline__ void scale_kv(unsigned char *stage, const float *f, int t, bool with_v = true) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (i >= 4 && !with_v) break;              // (the K tile is the first half of the stage)
        const int qi = t + CT * i;                 // 16-byte group index in the 64 KB stage
        const float fj = f[(qi & 1023) >> 3];      // row of this group (K and V tiles alike)
        uint4 v = *reinterpret_cast<const uint4 *>(stage + qi * 16);
        uint32_t *pv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
        for (int u = 0; u < 4; ++u) pv[u] = pack_bf16(bf16_lo(pv[u]) * fj, bf16_hi(pv[u]) * fj);
        *reinterpret_cast<uint4 *>(stage + qi * 16) = v;
    }
}

// ------------------------------------------------------------------------------------------------------------
// Segment summaries.  The weights are formed in log2 space from the run's total log-decay (one pre-pass over the
// gates) and a running prefix, so every tile is a pure accumulation into TMEM: no rescaling pass.  The kernel
// streams K and V once.  A summarised run never holds the last tile of its sequence, so all its tiles are full.
// ------------------------------------------------------------------------------------------------------------
enum { SB_KV0 = 0, SB_MMA = NS, SB_COUNT };

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
                const uint32_t kb = base14 + (uint32_t)(n % NS) * (STAGE >> 4), vb = kb + (32768u >> 4);
                if (n == 0) {
                    mma8_mm<0>(tm_H, kb, kb, kIdescMM);
                    mma8_mm<0>(tm_U, vb, kb, kIdescMM);
                } else {
                    mma8_mm<1>(tm_H, kb, kb, kIdescMM);
                    mma8_mm<1>(tm_U, vb, kb, kIdescMM);
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
            const uint32_t dst = sb + (uint32_t)(n % NS) * STAGE;
            const uint32_t bar = bars + 8 * (SB_KV0 + n % NS);
            mbar_expect_tx(bar, 65536u);
            tma_load_tile3(&tmK, dst, bar, h * a.d, tile_x_hi(h, a.d, a.heads), (n0 + n) * NT, b);
            tma_load_tile3(&tmV, dst + 32768, bar, h * a.d, tile_x_hi(h, a.d, a.heads), (n0 + n) * NT, b);
        };
        if (t == 0)
            for (int n = 0; n < ntiles && n < NS; ++n) issue_tma(n);

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
            return (t < NT && i < ntok_run) ? ldg_stream_f32(grun + (size_t)i * a.heads) : 1.f;
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
                // w_j = 2^(decay from token j to the end of the run) = 2^((total - prefix) - incl_j); its root scales the rows
                float wt = exp2f(0.5f * ((total - prefix) - incl));
                if (brun) wt *= sqrtf(fmaxf(__ldg(brun + (size_t)(n * NT + t) * a.heads), 0.f));   // write strength
                s_w[t] = wt;
                prefix += tile_total;
            }
            if (!mbar_spin_bounded(bars + 8 * (SB_KV0 + n % NS), (uint32_t)((n / NS) & 1))) s_abort = 1;
            asm volatile("bar.sync 1, 512;" ::: "memory");       // weights are published (and the scan scratch is free)
            scale_kv(smem + (size_t)(n % NS) * STAGE, s_w, t);
            fence_async_smem();
            if (t == 0) *reinterpret_cast<volatile int *>(&s_req) = n;
            asm volatile("bar.sync 3, 544;" ::: "memory");       // hand the tile to the issuing warp
            // the previous tile's products are done: its stage takes the tile after the next
            if (n >= 1) {
                if (!mbar_spin_bounded(bars + 8 * SB_MMA, (uint32_t)((n - 1) & 1))) s_abort = 1;
                if (t == 0 && n + 2 < ntiles) issue_tma(n + 2);
            }
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
// masters, which it keeps in registers in fp32 for a whole run.  The tensor cores compute only each tile's
// increments dH = K~^T K~, dU = V~^T K~ into one of two TMEM buffers, one tile ahead of their use; per tile a thread
// stores the bf16 copies of its part of the tile-initial H_0, U_0 (and adds up ||H_0||_F^2), then advances its
// masters: H <- zeta H + dH, U <- zeta U + dU.  The warp that issues the products also turns the gates into the row
// factors and the tile's decay, two tiles ahead, so that the compute warps meet no scan.  SPLIT: two blocks per work
// item, one keeps H (and loads only the keys), one keeps U.
// ------------------------------------------------------------------------------------------------------------
// TB_STG0 + stage: one barrier per stage, like the loads.  (With a single barrier the compute warps could complete two
// phases, tiles m + 1 and m + 2, while the TMA thread was still held up behind tile m's store; the phase parity it
// then polled looked incomplete, and the compute warps in turn waited for the load that only this thread issues.)
enum { TB_KV0 = 0, TB_D0 = NS, TB_D1, TB_STG0, TB_COUNT = TB_STG0 + NS };

template <bool SPLIT>
__global__ void __launch_bounds__(kThreadsStateK, 1)
fwd_tc_state_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const __grid_constant__ CUtensorMap tmS, FwdArgs a) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_bars[TB_COUNT];
    __shared__ uint32_t s_tmem_base;
    __shared__ float s_w[3][NT], s_red[3][16], s_decay[4];
    __shared__ int s_req, s_abort;
    unsigned char *smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    const uint32_t sb = smem_u32(smem), bars = smem_u32(&s_bars[0]);
    const int t = threadIdx.x, l = t & 31;
    // the solve kernel is launched as a programmatic dependent of this one
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (t == 0) {
        s_abort = 0;
        for (int i = 0; i < TB_COUNT; ++i)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bars + 8 * i), "r"(i >= TB_STG0 ? CT / 32 : 1));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (t < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&s_tmem_base))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = s_tmem_base;
    const WorkPlan &P = a.plan;
    // With no sequence cut and few work items the masters are split: two blocks per item, one advances H (and needs
    // only the keys), one U.  Each handles the masters w_lo <= which < w_hi.
    const int item = SPLIT ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int w_lo = SPLIT ? (int)(blockIdx.x & 1) : 0, w_hi = SPLIT ? w_lo + 1 : 2;
    const bool do_h = w_lo == 0, do_u = w_hi == 2;
    const long long f_lo = P.lo(item), f_hi = P.lo(item + 1);
    const int n_mine = (int)(f_hi - f_lo);
    const uint32_t base14 = (sb >> 4) & 0x3FFF;

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
    auto wait = [&](int which, uint32_t parity) {     // once a wait has given up the later ones return at once
        if (*reinterpret_cast<volatile int *>(&s_abort) == 0 && !mbar_spin_bounded(bars + 8 * which, parity))
            *reinterpret_cast<volatile int *>(&s_abort) = 1;
    };

    if (t >= CT + 32) {
        // ================================ TMA thread: loads of K, V; stores of the bf16 copies ================================
        if (l == 0 && n_mine > 0) {
            auto issue_tma = [&](int m) {
                const Pos p = pos_of(m);
                const uint32_t dst = sb + (uint32_t)(m % NS) * STAGE, bar = bars + 8 * (TB_KV0 + m % NS);
                mbar_expect_tx(bar, do_u ? 65536u : 32768u);
                tma_load_tile3(&tmK, dst, bar, p.h * a.d, tile_x_hi(p.h, a.d, a.heads), p.n * NT, p.b);
                if (do_u) tma_load_tile3(&tmV, dst + 32768, bar, p.h * a.d, tile_x_hi(p.h, a.d, a.heads), p.n * NT, p.b);
            };
            for (int m = 0; m < n_mine && m < NS; ++m) issue_tma(m);
            for (int m = 0; m < n_mine; ++m) {
                // the compute warps have written the bf16 copies of H_0, U_0 over the tile's K and V (the tile's
                // products are complete): store them, then the stage takes the tile three further on
                wait(TB_STG0 + m % NS, (uint32_t)((m / NS) & 1));
                const uint32_t src = sb + (uint32_t)(m % NS) * STAGE;
                for (int which = w_lo; which < w_hi; ++which)
                    for (int hf = 0; hf < 2; ++hf)
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::
                                         "l"(reinterpret_cast<uint64_t>(&tmS)), "r"(64 * hf), "r"((int)((f_lo + m) * 256 + 128 * which)),
                                     "r"(src + 32768 * which + 16384 * hf)
                                     : "memory");
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                if (m + NS < n_mine) {
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the copies have been read
                    issue_tma(m + NS);
                }
            }
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");    // the stores are complete
        }
    } else if (t >= CT) {
        // ================ MMA issuing warp; it also prepares the row factors, two tiles ahead ================
        // Row factors sqrt(beta_j 2^(G_last - G_j)) (0 past the sequence) and decay of tile m: lane l has tokens l, 32 + l,
        // 64 + l, 96 + l.  Written two hand-overs before the compute warps read them, so the hand-over barrier in between
        // orders the two; three sets, so that no set is rewritten while a slower warp may still read it.
        float lg[4], sb[4];          // gates and write strengths of the tile whose factors come next (loaded a hand-over ahead)
        auto load_scalars = [&](int m, float(&lg)[4], float(&sb)[4]) {
#pragma unroll
            for (int grp = 0; grp < 4; ++grp) {
                lg[grp] = 1.f;
                sb[grp] = 0.f;
            }
            if (m >= n_mine) return;
            const Pos p = pos_of(m);
#pragma unroll
            for (int grp = 0; grp < 4; ++grp) {
                const int tok = 32 * grp + l;
                if (tok < p.ntok) {
                    lg[grp] = ldg_stream_f32(a.gate + p.tok0 + (size_t)tok * a.heads);
                    sb[grp] = a.beta ? fmaxf(ldg_stream_f32(a.beta + p.tok0 + (size_t)tok * a.heads), 0.f) : 1.f;
                }
            }
        };
        auto factors = [&](int m, float(&lg)[4], const float(&sb)[4]) {      // from the loaded scalars of tile m
            float before = 0.f;
#pragma unroll
            for (int grp = 0; grp < 4; ++grp) {
                float incl = fmaxf(log2f(lg[grp]), -115.f);
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const float up = __shfl_up_sync(0xffffffffu, incl, o);
                    if (l >= o) incl += up;
                }
                const float tot = __shfl_sync(0xffffffffu, incl, 31);
                lg[grp] = incl + before;             // cumulative log2 gate up to and including the token
                before += tot;
            }
            const float tile_total = before;
#pragma unroll
            for (int grp = 0; grp < 4; ++grp) s_w[m % 3][32 * grp + l] = sqrtf(sb[grp]) * exp2f(0.5f * (tile_total - lg[grp]));
            if (l == 0) s_decay[m & 3] = exp2f(tile_total);      // (four deep: tile m's is read after the hand-over of tile m + 1, behind which tile m + 3's is written)
            __syncwarp();
        };
        if (n_mine > 0) {
            float lg1[4], sb1[4];
            load_scalars(0, lg, sb);
            load_scalars(1, lg1, sb1);               // (both tiles' loads in flight together)
            factors(0, lg, sb);
            if (n_mine > 1) factors(1, lg1, sb1);
            load_scalars(2, lg, sb);
            asm volatile("bar.sync 3, 544;" ::: "memory");       // the factors of the first two tiles are published
        }
        for (;;) {
            asm volatile("bar.sync 3, 544;" ::: "memory");
            const int m = *reinterpret_cast<const volatile int *>(&s_req);
            if (m < 0) break;
            if (l == 0) {
                fence_after();
                const uint32_t kb = base14 + (uint32_t)(m % NS) * (STAGE >> 4), vb = kb + (32768u >> 4);
                const uint32_t tm_d = tmem + 256 * (m & 1);
                if (do_h) mma8_mm<0>(tm_d, kb, kb, kIdescMM);              // dH = K~^T K~
                if (do_u) mma8_mm<0>(tm_d + 128, vb, kb, kIdescMM);        // dU = V~^T K~
                mma_commit(bars + 8 * (TB_D0 + (m & 1)));
            }
            __syncwarp();
            if (m + 2 < n_mine) {
                factors(m + 2, lg, sb);
                load_scalars(m + 3, lg, sb);         // (in flight across the hand-over)
            }
        }
    } else if (n_mine > 0) {
        // ================================= compute threads =================================
        const int q = (t >> 5) & 3, cq = t >> 7, c = 32 * q + l;
        const uint32_t lane_addr = (uint32_t)(32 * q) << 16;
        const size_t st = state_floats(D, D);
        // first item of the chain of summaries behind this block's start state
        int chain_j0 = item;
        if (P.cut_in(item)) {
            const long long seq_start = (f_lo / P.N) * P.N;
            chain_j0 = item - 1;
            while (P.lo(chain_j0) > seq_start) --chain_j0;
        }
        // Tile m: rows scaled in place by the row factors (prepared by the issuing warp), products posted.
        auto prepare = [&](int m) {
            wait(TB_KV0 + m % NS, (uint32_t)((m / NS) & 1));
            scale_kv(smem + (size_t)(m % NS) * STAGE, s_w[m % 3], t, do_u);
            fence_async_smem();
            fence_before();
            if (t == 0) *reinterpret_cast<volatile int *>(&s_req) = m;
            asm volatile("bar.sync 3, 544;" ::: "memory");       // hand the tile to the issuing warp
        };

        float mH[32], mU[32];
        asm volatile("bar.sync 3, 544;" ::: "memory");           // the factors of the first two tiles are published
        prepare(0);
        // summaries and start states are read after this point only
        asm volatile("griddepcontrol.wait;" ::: "memory");

        for (int m = 0; m < n_mine; ++m) {
            const Pos p = pos_of(m);
            if (m + 1 < n_mine) prepare(m + 1);                  // its products run under this tile's passes
            const long long tile = f_lo + m;
            if (p.run_start) {
                // start of a run: the caller's initial state of the sequence (or zero), carried through the summaries
                // of the blocks that hold the earlier part of the sequence: state <- decay_j * state + delta_j
                const bool chained = p.n != 0;
                const float *s0 = (chained && a.start_from_scan) ? a.ws.start + (size_t)item * st
                                  : (a.state_in ? a.state_in + (size_t)p.seq * st : nullptr);
                const int j0 = (chained && !a.start_from_scan) ? chain_j0 : 0, j1 = (chained && !a.start_from_scan) ? item : 0;
                const size_t e = (size_t)c * D + 32 * cq;
                // the caller's state has head dimension a.d (rows and columns from a.d on are zero on chip); the scan
                // kernel's start states are in the on-chip layout
                const bool ext = s0 != nullptr && !(chained && a.start_from_scan);
                const float *const s0e = ext ? a.state_in + (size_t)p.seq * 2 * a.d * a.d + (size_t)c * a.d + 32 * cq : nullptr;
                const bool in_ext = c < a.d && 32 * cq < a.d;
#pragma unroll
                for (int which = 0; which < 2; ++which) {
                    if (which < w_lo || which >= w_hi) continue;
                    float(&mm)[32] = which ? mU : mH;
                    const size_t eo = e + which * (size_t)D * D;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float4 v4 = ext ? (in_ext ? *reinterpret_cast<const float4 *>(s0e + which * (size_t)a.d * a.d + 4 * i)
                                                        : make_float4(0.f, 0.f, 0.f, 0.f))
                                          : (s0 ? *reinterpret_cast<const float4 *>(s0 + eo + 4 * i) : make_float4(0.f, 0.f, 0.f, 0.f));
                        mm[4 * i + 0] = v4.x; mm[4 * i + 1] = v4.y; mm[4 * i + 2] = v4.z; mm[4 * i + 3] = v4.w;
                    }
                    for (int j = j0; j < j1; ++j) {
                        // summaries come from the kernel this one may overlap with as its programmatic dependent: ordinary loads
                        const float dj = *reinterpret_cast<const volatile float *>(a.ws.decay + j);
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float4 dd = *(reinterpret_cast<const float4 *>(a.ws.delta + (size_t)j * st + eo) + i);
                            mm[4 * i + 0] = fmaf(dj, mm[4 * i + 0], dd.x);
                            mm[4 * i + 1] = fmaf(dj, mm[4 * i + 1], dd.y);
                            mm[4 * i + 2] = fmaf(dj, mm[4 * i + 2], dd.z);
                            mm[4 * i + 3] = fmaf(dj, mm[4 * i + 3], dd.w);
                        }
                    }
                }
            }
            // ---- bf16 copies of the tile-initial state and ||H_0||_F^2: each master in turn is written over the tile's
            // own K (V) in operand layout and goes from there to the workspace by TMA; then its increments are added
            wait(TB_D0 + (m & 1), (uint32_t)((m >> 1) & 1));     // the tile's increments are complete (posted a tile ago)
            fence_after();
            const float decay = s_decay[m & 3];
            unsigned char *const stg = smem + (size_t)(m % NS) * STAGE;   // the tile's own K and V are no longer needed
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                if (which < w_lo || which >= w_hi) continue;
                float(&mm)[32] = which ? mU : mH;
                float hs = 0.f;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint32_t pk[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float v0 = mm[8 * i + 2 * u], v1 = mm[8 * i + 2 * u + 1];
                        if (which == 0) hs = fmaf(v0, v0, fmaf(v1, v1, hs));
                        pk[u] = pack_bf16(v0, v1);
                    }
                    *reinterpret_cast<uint4 *>(stg + 32768 * which + tile_off(c, 4 * cq + i)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
                if (which == 0) {
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) hs += __shfl_xor_sync(0xffffffffu, hs, o);
                    if (l == 0) s_red[m % 3][t >> 5] = hs;
                }
                if (which == w_hi - 1) {
                    fence_async_smem();
                    __syncwarp();
                    if (l == 0) mbar_arrive(bars + 8 * (TB_STG0 + m % NS));  // -> the TMA thread stores both copies
                }
                // advance the master: zeta m + increment
#pragma unroll
                for (int piece = 0; piece < 2; ++piece) {
                    uint32_t r[16];
                    TMEM_LD16(tmem + 256 * (m & 1) + 128 * which + lane_addr + 32 * cq + 16 * piece, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; ++i) mm[16 * piece + i] = fmaf(decay, mm[16 * piece + i], __uint_as_float(r[i]));
                }
            }
            fence_before();
            // ---- final state of the sequence
            if (p.seq_end && a.state_out && c < a.d && 32 * cq < a.d) {      // in the caller's layout (head dimension a.d)
                float *so = a.state_out + (size_t)p.seq * 2 * a.d * a.d + (size_t)c * a.d + 32 * cq;
#pragma unroll
                for (int which = 0; which < 2; ++which) {
                    if (which < w_lo || which >= w_hi) continue;
                    const float(&mm)[32] = which ? mU : mH;
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        *reinterpret_cast<float4 *>(so + which * (size_t)a.d * a.d + 4 * i) = make_float4(mm[4 * i], mm[4 * i + 1], mm[4 * i + 2], mm[4 * i + 3]);
                }
            }
            // ||H_0||_F^2 of the previous tile: its per-warp sums were written before this tile's hand-over barrier (the
            // block's last tile has none: the sums of the last two tiles are read after the loop).  Three sets of sums,
            // so that a warp that runs a tile ahead writes none that is still to be read.
            if (t == 0 && m >= 1 && m + 1 < n_mine && do_h) {
                float hh = 0.f;
#pragma unroll
                for (int i = 0; i < 16; ++i) hh += s_red[(m - 1) % 3][i];
                a.tile_hh[tile - 1] = hh;
            }
        }
        if (t == 0) *reinterpret_cast<volatile int *>(&s_req) = -1;
        asm volatile("bar.sync 3, 544;" ::: "memory");           // releases the issuing warp; the last sums are published
        if (t == 0) {
            for (int m = n_mine >= 2 ? n_mine - 2 : n_mine - 1; m < n_mine && do_h; ++m) {
                float hh = 0.f;
#pragma unroll
                for (int i = 0; i < 16; ++i) hh += s_red[m % 3][i];
                a.tile_hh[f_lo + m] = hh;
            }
            if (s_abort != 0 && a.device_status) atomicExch(a.device_status, (int)GKA_ERR_TIMEOUT);
        }
    } else {
        if (t == 0) *reinterpret_cast<volatile int *>(&s_req) = -1;
        asm volatile("bar.sync 3, 544;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    if (t < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
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
    int sms_here = 0, dev_here = 0;
    if ((err = cudaGetDevice(&dev_here)) != cudaSuccess) return err;
    if ((err = cudaDeviceGetAttribute(&sms_here, cudaDevAttrMultiProcessorCount, dev_here)) != cudaSuccess) return err;
    // two blocks per work item (one per master) where no sequence is cut and the blocks still fit one per SM
    a.state_split = (!any_cut && 2 * a.plan.G <= sms_here) ? 1 : 0;
    alignas(64) CUtensorMap tmK, tmV, tmS;      // boxes of 128 tokens x 64 channels; per-tile bf16 state copies
    const int cols = a.heads * a.d;
    if (!make_tile_map(&tmK, a.k, a.B, a.T, cols, NT) || !make_tile_map(&tmV, a.v, a.B, a.T, cols, NT) ||
        !make_state_map(&tmS, a.tile_hu, (unsigned long long)a.plan.NC * 256ull))
        return cudaErrorInvalidValue;
    if (any_cut) {
        err = cudaFuncSetAttribute(fwd_tc_summary_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)KV_SMEM);
        if (err != cudaSuccess) return err;
        fwd_tc_summary_kernel<<<a.plan.G, kThreadsState, KV_SMEM, stream>>>(tmK, tmV, a);
        if (a.start_from_scan) {
            err = launch_fwd_scan(a, (int)state_floats(D, D), stream, true);
            if (err != cudaSuccess) return err;
        }
        a.after_summary = 1;
    }
    auto state_kernel = a.state_split ? fwd_tc_state_kernel<true> : fwd_tc_state_kernel<false>;
    err = cudaFuncSetAttribute(state_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ST_SMEM);
    if (err != cudaSuccess) return err;
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(a.plan.G * (a.state_split ? 2 : 1)));
        cfg.blockDim = dim3(kThreadsStateK);
        cfg.dynamicSmemBytes = ST_SMEM;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = a.after_summary ? 1 : 0;
        err = cudaLaunchKernelEx(&cfg, state_kernel, tmK, tmV, tmS, a);
        if (err != cudaSuccess) return err;
    }
    return launch_fwd_solve(a, stream);
}

}  // namespace gka
