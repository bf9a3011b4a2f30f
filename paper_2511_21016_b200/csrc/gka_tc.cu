// tcgen05 path of the chunked GKA forward (bf16 operands, fp32 accumulation) for sm_100a: launcher and the
// segment-summary kernel.  The main kernel (token-major tiles, Chebyshev solve) is in gka_tc_tile.cu.
//
// Segment summaries: for every work item whose range ends inside a sequence (gka_common.cuh explains the work
// decomposition), the decay product and (delta-H, delta-U) of its last run, i.e. the run's final state for a
// zero start state (the state recurrences of Section 3 / 4.2.1 unrolled over the run):
//     dH = sum_j w_j k_j k_j^T,   dU = sum_j w_j v_j k_j^T,   w_j = product of the gates after token j in the run.
// The weights are formed in log2 space from the run's total log-decay (one pre-pass over the gates) and a
// running prefix, so every tile of 128 tokens is a pure accumulation K^T (w o K), V^T (w o K) into TMEM: no
// rescaling pass.  The kernel streams K and V once (it is bound by HBM): three TMA stages of K and V tiles
// keep two tiles in flight while the third is consumed; one extra warp issues the products.
#include <cuda.h>

#include "gka_common.cuh"
#include "gka_tc_util.cuh"

namespace gka {
cudaError_t launch_fwd_tile(const FwdArgs &a, cudaStream_t stream);
namespace {

using namespace tcu;

constexpr int D = 128;
constexpr int C = kChunk;
constexpr int NT = 128;                                  // tokens per tile
constexpr int SUM_CT = 512;                              // compute threads; + one warp that issues the products
constexpr int SUM_NS = 3;                                // TMA stages
constexpr uint32_t SUM_STAGE = 65536;                    // K tile + V tile, [128 rows][128 channels] bf16 each
constexpr uint32_t SUM_OFF_KW = SUM_NS * SUM_STAGE;      // w o K
constexpr uint32_t SUM_SMEM = SUM_OFF_KW + 32768 + 1024; // + slack for the 1024-byte alignment of the base
enum { SB_KV0 = 0, SB_MMA = SUM_NS, SB_COUNT };

__global__ void __launch_bounds__(SUM_CT + 32, 1)
fwd_tc_summary_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, FwdArgs a) {
    const WorkPlan &P = a.plan;
    const int item = blockIdx.x;
    // the main kernel may be launched as a programmatic dependent: its blocks may take the SMs that this grid leaves
    // and run their prologue; they wait for this grid's completion before they read a summary
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
    const int nch = (int)(f1 - f0);
    const int ntiles = (nch + 1) / 2;

    if (t >= SUM_CT) {
        // ================================ MMA issuing warp ================================
        constexpr uint32_t I_MM = make_idesc(128, 128, 1, 1);      // both operands MN-major
        for (;;) {
            asm volatile("bar.sync 3, 544;" ::: "memory");         // the compute threads hand over a tile
            const int n = *reinterpret_cast<const volatile int *>(&s_req);
            if (n < 0) break;
            if (l == 0) {
                fence_after();
                const uint32_t st0 = sb + (uint32_t)(n % SUM_NS) * SUM_STAGE;
                const uint32_t k_mn = desc_lo(st0, 16384), v_mn = desc_lo(st0 + 32768, 16384);
                const uint32_t kw_mn = desc_lo(sb + SUM_OFF_KW, 16384);
                if (n == 0) {
                    mma_ss_r<0>(tm_H, k_mn, 0, kw_mn, 0, I_MM);
                    mma_ss_r<0>(tm_U, v_mn, 0, kw_mn, 0, I_MM);
                } else {
                    mma_ss_r<1>(tm_H, k_mn, 0, kw_mn, 0, I_MM);
                    mma_ss_r<1>(tm_U, v_mn, 0, kw_mn, 0, I_MM);
                }
#pragma unroll
                for (int ks = 1; ks < 8; ++ks) {
                    mma_ss_r<1>(tm_H, k_mn, mnstep(ks), kw_mn, mnstep(ks), I_MM);
                    mma_ss_r<1>(tm_U, v_mn, mnstep(ks), kw_mn, mnstep(ks), I_MM);
                }
                mma_commit(bars + 8 * SB_MMA);
            }
            __syncwarp();
        }
    } else {
        // ================================= compute threads =================================
        const int seq = (int)((unsigned)f0 / (unsigned)P.N), b = seq / a.heads, h = seq % a.heads;
        const int n0 = (int)((unsigned)f0 - (unsigned)seq * (unsigned)P.N);   // first chunk of the run in its sequence
        const float *grun = a.gate + ((size_t)b * a.T + (size_t)n0 * C) * a.heads + h;   // token stride: heads
        const float *brun = a.beta ? a.beta + ((size_t)b * a.T + (size_t)n0 * C) * a.heads + h : nullptr;
        const int ntok_run = nch * C;
        auto issue_tma = [&](int n) {
            const uint32_t dst = sb + (uint32_t)(n % SUM_NS) * SUM_STAGE;
            const int y = (n0 + 2 * n) * C;
            const uint32_t bar = bars + 8 * (SB_KV0 + n % SUM_NS);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(65536u) : "memory");
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int x = h * D + 64 * hf;
                asm volatile(
                    "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::
                        "r"(dst + 16384 * hf), "l"(reinterpret_cast<uint64_t>(&tmK)), "r"(x), "r"(y), "r"(b), "r"(bar)
                    : "memory");
                asm volatile(
                    "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::
                        "r"(dst + 32768 + 16384 * hf), "l"(reinterpret_cast<uint64_t>(&tmV)), "r"(x), "r"(y), "r"(b), "r"(bar)
                    : "memory");
            }
        };
        if (t == 0)
            for (int n = 0; n < ntiles && n < SUM_NS; ++n) issue_tma(n);

        // ---- pre-pass: total log2 decay of the run
        float total = 0.f;
        {
            float s = 0.f;
            for (int i0 = t; i0 < ntok_run; i0 += 4 * SUM_CT) {     // four independent loads in flight per thread
                float g[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = i0 + u * SUM_CT;
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

        // threads 0..127: gate of token t of tile n (1 past the run); fetched one tile ahead, the logarithm is
        // taken when the value is used so that nothing waits for the load
        auto load_gate = [&](int n) -> float {
            const int i = n * NT + t;
            return (t < NT && i < ntok_run) ? __ldg(grun + (size_t)i * a.heads) : 1.f;
        };
        float g_cur = load_gate(0);
        float prefix = 0.f;                    // log2 decay of the tiles before the current one
        for (int n = 0; n < ntiles; ++n) {
            const float g_next = load_gate(n + 1);
            // inclusive prefix of the tile's log2 gates (threads 0..127), weights of the tile's tokens
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
                // w_j = 2^(decay from token j to the end of the run) = 2^((total - prefix) - incl_j); 0 past the run
                float wt = (n * NT + t < ntok_run) ? exp2f((total - prefix) - incl) : 0.f;
                if (brun && n * NT + t < ntok_run) wt *= fmaxf(__ldg(brun + (size_t)(n * NT + t) * a.heads), 0.f);   // write strength
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
                const int qi = t + SUM_CT * i;             // 16-byte group index in the 32 KB tile
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
    // Short chains are folded by the main kernel's blocks themselves; long ones (a sequence spread over many
    // work items) would make every block re-read its whole chain, so the scan kernel materialises the start
    // states once instead.
    a.start_from_scan = longest > 4 ? 1 : 0;
    if (any_cut) {
        alignas(64) CUtensorMap tmK, tmV;      // boxes of 128 tokens x 64 channels
        const int cols = a.heads * D;
        if (!make_tile_map(&tmK, a.k, a.B, a.T, cols, NT) || !make_tile_map(&tmV, a.v, a.B, a.T, cols, NT))
            return cudaErrorInvalidValue;
        err = cudaFuncSetAttribute(fwd_tc_summary_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SUM_SMEM);
        if (err != cudaSuccess) return err;
        fwd_tc_summary_kernel<<<a.plan.G, SUM_CT + 32, SUM_SMEM, stream>>>(tmK, tmV, a);
        if (a.start_from_scan) {
            err = launch_fwd_scan(a, (int)state_floats(D, D), stream, true);
            if (err != cudaSuccess) return err;
        }
        a.after_summary = 1;     // the main kernel follows its producer (summary or scan kernel) as a programmatic dependent
    }
    return launch_fwd_tile(a, stream);
}

}  // namespace gka
