// Recurrent GKA step over a few consecutive tokens (eq. (CH) applied token after token per (sequence, head))
// for sm_100a: speculative / multi-token decoding.  Same organisation as the single-token kernel
// (gka_decode.cu) - H in registers, U in shared memory, one block of 256 threads per (sequence, head) - but
// the state is read once before the first token and written once after the last, so its HBM traffic is
// shared by all tokens of the call.
#include "gka_common.cuh"

namespace gka {
namespace {

constexpr int kThreadsMulti = 256;

template <int D, typename IoT>
__global__ void __launch_bounds__(kThreadsMulti, 2)
decode_multi_kernel(float *__restrict__ state, const IoT *__restrict__ q, const IoT *__restrict__ k,
                    const IoT *__restrict__ v, const float *__restrict__ gate, const float *__restrict__ lam,
                    int n_iter, IoT *__restrict__ out, unsigned flags, const float *__restrict__ beta,
                    const float *__restrict__ alpha, int T, int heads, int *__restrict__ device_status) {
    constexpr int RPT = D / 32;   // rows per thread
    constexpr int CG = D / 32;    // float4 column groups per thread
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float *sU = reinterpret_cast<float *>(smem_raw);          // [D][D] U, updated in place token after token
    float *sX = sU + D * D;                                   // [2][D] iterate, double-buffered
    float *sQ = sX + 2 * D;                                   // [D]
    float *sKv = sQ + D;                                      // [D] k
    float *sVv = sKv + D;                                     // [D] v
    float *sRed = sVv + D;                                    // [16]
    uint64_t *bar = reinterpret_cast<uint64_t *>(sRed + 16);

    const int sh = blockIdx.x;                                // (sequence, head) pair
    const int seq = sh / heads, h = sh % heads;
    const int tid = threadIdx.x, lane8 = tid & 7, rgrp = tid >> 3;
    float *gH = state + (size_t)sh * (2 * D * D);
    float *gU = gH + D * D;

    // ---- kick off the bulk copy of U
    const uint32_t bar_addr = smem_u32(bar);
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_addr));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) {
        constexpr uint32_t bytes = D * D * sizeof(float);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_addr), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
                         "r"(smem_u32(sU)), "l"(gU), "r"(bytes), "r"(bar_addr)
                     : "memory");
    }

    // ---- H into registers
    float4 Hr[RPT][CG];
#pragma unroll
    for (int m = 0; m < RPT; ++m)
#pragma unroll
        for (int n = 0; n < CG; ++n)
            Hr[m][n] = __ldcs(reinterpret_cast<const float4 *>(gH + (size_t)(rgrp + 32 * m) * D + 4 * (lane8 + 8 * n)));

    for (int t = 0; t < T; ++t) {
        const size_t tok = ((size_t)seq * T + t) * heads + h;
        if (tid < D) {
            // write strength beta (Remark on the beta-augmented variant, Section 4.1): beta k k^T and beta v k^T are
            // the plain writes of sqrt(beta) k and sqrt(beta) v
            const float sb = beta ? sqrtf(fmaxf(beta[tok], 0.f)) : 1.f;
            sQ[tid] = Io<IoT>::load1(q + tok * D + tid);
            sKv[tid] = sb * Io<IoT>::load1(k + tok * D + tid);
            sVv[tid] = sb * Io<IoT>::load1(v + tok * D + tid);
        }
        const float gam = gate[tok];
        float lamv = lam[tok];
        const float al = alpha ? alpha[tok] : 1.f;   // alpha-connection (Section 4.3): the read uses alpha x + (1 - alpha) q
        __syncthreads();

        // ---- H <- gamma H + k k^T (kept in registers), Frobenius norm
        float kc[CG][4], kr[RPT];
#pragma unroll
        for (int n = 0; n < CG; ++n) {
            float4 t4 = *reinterpret_cast<const float4 *>(sKv + 4 * (lane8 + 8 * n));
            kc[n][0] = t4.x; kc[n][1] = t4.y; kc[n][2] = t4.z; kc[n][3] = t4.w;
        }
#pragma unroll
        for (int m = 0; m < RPT; ++m) kr[m] = sKv[rgrp + 32 * m];
        float ss = 0.f;
#pragma unroll
        for (int m = 0; m < RPT; ++m)
#pragma unroll
            for (int n = 0; n < CG; ++n) {
                float4 h4 = Hr[m][n];
                h4.x = fmaf(gam, h4.x, kr[m] * kc[n][0]);
                h4.y = fmaf(gam, h4.y, kr[m] * kc[n][1]);
                h4.z = fmaf(gam, h4.z, kr[m] * kc[n][2]);
                h4.w = fmaf(gam, h4.w, kr[m] * kc[n][3]);
                Hr[m][n] = h4;
                ss += h4.x * h4.x + h4.y * h4.y + h4.z * h4.z + h4.w * h4.w;
                // the last token's H is final: it goes back at once, under the iterations that follow
                if (t == T - 1) __stcs(reinterpret_cast<float4 *>(gH + (size_t)(rgrp + 32 * m) * D + 4 * (lane8 + 8 * n)), h4);
            }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if ((tid & 31) == 0) sRed[tid >> 5] = ss;
        __syncthreads();
        float fro2 = 0.f;
#pragma unroll
        for (int i = 0; i < kThreadsMulti / 32; ++i) fro2 += sRed[i];
        const float fro = sqrtf(fro2);
        if (flags & GKA_FLAG_ADAPTIVE_LAMBDA) lamv *= fro;

        // ---- Algorithm 1, L = fro + lambda, mu = lambda
        const float Lpm = fro + 2.f * lamv;
        const float rho = fro / Lpm, rho2 = rho * rho, s0 = 2.f / Lpm;
        float omega = 2.f;
        // Row sums of the matvec are reduced across the 8 lanes of a row group so that each lane pair ends up with
        // one of the group's RPT rows (a transposing butterfly: fewer shuffles than RPT full reductions, and every
        // row's update is computed by two lanes instead of eight).  Lane pair p = lane8 >> 1 owns row rgrp + 32 p.
        static_assert(RPT == 4 || RPT == 2, "row ownership below assumes 2 or 4 rows per thread");
        const int myrow = rgrp + 32 * (RPT == 4 ? (lane8 >> 1) : (lane8 >> 2));
        const float qr = sQ[myrow];
        float xr = s0 * qr, xpr = 0.f;
        if ((RPT == 4 ? (lane8 & 1) : (lane8 & 3)) == 0) sX[myrow] = xr;
        __syncthreads();
        int cur = 0;
        for (int it = 0; it < n_iter; ++it) {
            const float *xs = sX + cur * D;
            float xc[CG][4];
#pragma unroll
            for (int n = 0; n < CG; ++n) {
                float4 t4 = *reinterpret_cast<const float4 *>(xs + 4 * (lane8 + 8 * n));
                xc[n][0] = t4.x; xc[n][1] = t4.y; xc[n][2] = t4.z; xc[n][3] = t4.w;
            }
            omega = 4.f / (4.f - rho2 * omega);
            const float step = s0 * omega, mom = omega - 1.f;
            float sm[RPT];
#pragma unroll
            for (int m = 0; m < RPT; ++m) {
                float s = 0.f;
#pragma unroll
                for (int n = 0; n < CG; ++n) {
                    s = fmaf(Hr[m][n].x, xc[n][0], s);
                    s = fmaf(Hr[m][n].y, xc[n][1], s);
                    s = fmaf(Hr[m][n].z, xc[n][2], s);
                    s = fmaf(Hr[m][n].w, xc[n][3], s);
                }
                sm[m] = s;
            }
            float tot;
            if (RPT == 4) {
                const bool hi4 = (lane8 & 4) != 0, hi2 = (lane8 & 2) != 0;
                float a0 = hi4 ? sm[2] : sm[0], a1 = hi4 ? sm[RPT - 1] : sm[1];
                a0 += __shfl_xor_sync(0xffffffffu, hi4 ? sm[0] : sm[2], 4);
                a1 += __shfl_xor_sync(0xffffffffu, hi4 ? sm[1] : sm[RPT - 1], 4);
                tot = (hi2 ? a1 : a0) + __shfl_xor_sync(0xffffffffu, hi2 ? a0 : a1, 2);
                tot += __shfl_xor_sync(0xffffffffu, tot, 1);
            } else {
                const bool hi4 = (lane8 & 4) != 0;
                tot = (hi4 ? sm[1] : sm[0]) + __shfl_xor_sync(0xffffffffu, hi4 ? sm[0] : sm[1], 4);
                tot += __shfl_xor_sync(0xffffffffu, tot, 2);
                tot += __shfl_xor_sync(0xffffffffu, tot, 1);
            }
            const float y = fmaf(lamv, xr, tot);
            const float xn = xr - step * (y - qr) + mom * (xr - xpr);
            xpr = xr;
            xr = xn;
            if ((RPT == 4 ? (lane8 & 1) : (lane8 & 3)) == 0) sX[(cur ^ 1) * D + myrow] = xn;
            cur ^= 1;
            __syncthreads();
        }

        // ---- (first token) wait for U (bounded); U <- gamma U + v k^T in place, output o = gamma (U_old x) + v (k . x)
        if (t == 0 && !mbar_wait_bounded(bar_addr, 0u)) {   // the copy never landed: leave the state untouched
            if (tid == 0 && device_status) atomicExch(device_status, (int)GKA_ERR_TIMEOUT);
            return;
        }
        const float *xs = sX + cur * D;
        float xc[CG][4];
        float kx = 0.f;
#pragma unroll
        for (int n = 0; n < CG; ++n) {
            float4 t4 = *reinterpret_cast<const float4 *>(xs + 4 * (lane8 + 8 * n));
            if (alpha) {
                const float4 q4 = *reinterpret_cast<const float4 *>(sQ + 4 * (lane8 + 8 * n));
                t4.x = fmaf(al, t4.x - q4.x, q4.x); t4.y = fmaf(al, t4.y - q4.y, q4.y);
                t4.z = fmaf(al, t4.z - q4.z, q4.z); t4.w = fmaf(al, t4.w - q4.w, q4.w);
            }
            xc[n][0] = t4.x; xc[n][1] = t4.y; xc[n][2] = t4.z; xc[n][3] = t4.w;
#pragma unroll
            for (int u = 0; u < 4; ++u) kx = fmaf(kc[n][u], xc[n][u], kx);
        }
        kx += __shfl_xor_sync(0xffffffffu, kx, 1);
        kx += __shfl_xor_sync(0xffffffffu, kx, 2);
        kx += __shfl_xor_sync(0xffffffffu, kx, 4);
#pragma unroll
        for (int m = 0; m < RPT; ++m) {
            const int row = rgrp + 32 * m;
            const float vr = sVv[row];
            float s = 0.f;
#pragma unroll
            for (int n = 0; n < CG; ++n) {
                float4 *pu = reinterpret_cast<float4 *>(sU + row * D + 4 * (lane8 + 8 * n));   // this thread's own elements
                float4 u4 = *pu;
                s = fmaf(u4.x, xc[n][0], s);
                s = fmaf(u4.y, xc[n][1], s);
                s = fmaf(u4.z, xc[n][2], s);
                s = fmaf(u4.w, xc[n][3], s);
                u4.x = fmaf(gam, u4.x, vr * kc[n][0]);
                u4.y = fmaf(gam, u4.y, vr * kc[n][1]);
                u4.z = fmaf(gam, u4.z, vr * kc[n][2]);
                u4.w = fmaf(gam, u4.w, vr * kc[n][3]);
                if (t == T - 1) __stcs(reinterpret_cast<float4 *>(gU + (size_t)row * D + 4 * (lane8 + 8 * n)), u4);   // final U
                else *pu = u4;
            }
            s += __shfl_xor_sync(0xffffffffu, s, 1);
            s += __shfl_xor_sync(0xffffffffu, s, 2);
            s += __shfl_xor_sync(0xffffffffu, s, 4);
            if (lane8 == 0) Io<IoT>::store1(out + tok * D + row, fmaf(gam, s, vr * kx));
        }
        __syncthreads();      // the token's vectors and iterate buffers are free for the next token
    }

}

template <int D, typename IoT>
cudaError_t launch_multi_typed(float *state, const void *q, const void *k, const void *v, const float *gate,
                               const float *lam, int n_iter, void *out, int nseq, int T, int heads, unsigned flags,
                               const float *beta, const float *alpha, int *device_status, cudaEvent_t ev_start,
                               cudaEvent_t ev_stop, cudaStream_t stream) {
    const size_t smem = (size_t)(D * D + 5 * D + 16) * sizeof(float) + 16;
    cudaError_t err = cudaFuncSetAttribute(decode_multi_kernel<D, IoT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    if (ev_start) cudaEventRecord(ev_start, stream);
    decode_multi_kernel<D, IoT><<<nseq * heads, kThreadsMulti, smem, stream>>>(
        state, reinterpret_cast<const IoT *>(q), reinterpret_cast<const IoT *>(k), reinterpret_cast<const IoT *>(v),
        gate, lam, n_iter, reinterpret_cast<IoT *>(out), flags, beta, alpha, T, heads, device_status);
    if (ev_stop) cudaEventRecord(ev_stop, stream);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode_multi(float *state, const void *q, const void *k, const void *v, const float *gate,
                                const float *lam, int n_iter, void *out, int nseq, int T, int heads, int d, int io_dtype,
                                unsigned flags, const float *beta, const float *alpha, int *device_status,
                                cudaEvent_t ev_start, cudaEvent_t ev_stop, cudaStream_t stream) {
    if (d == 128)
        return io_dtype == GKA_BF16
                   ? launch_multi_typed<128, __nv_bfloat16>(state, q, k, v, gate, lam, n_iter, out, nseq, T, heads, flags, beta, alpha, device_status, ev_start, ev_stop, stream)
                   : launch_multi_typed<128, float>(state, q, k, v, gate, lam, n_iter, out, nseq, T, heads, flags, beta, alpha, device_status, ev_start, ev_stop, stream);
    return io_dtype == GKA_BF16
               ? launch_multi_typed<64, __nv_bfloat16>(state, q, k, v, gate, lam, n_iter, out, nseq, T, heads, flags, beta, alpha, device_status, ev_start, ev_stop, stream)
               : launch_multi_typed<64, float>(state, q, k, v, gate, lam, n_iter, out, nseq, T, heads, flags, beta, alpha, device_status, ev_start, ev_stop, stream);
}

}  // namespace gka
