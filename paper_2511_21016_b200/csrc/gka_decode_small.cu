// Recurrent GKA step (eq. (CH) applied token after token) for the small head dimensions 16 and 32 on sm_100a: one
// warp per (sequence, head) pair.  Lane l keeps row l of H and row l of U in registers (2 D floats), a vector is one
// element per lane, and every matrix-vector product is D shuffles and D FMAs per lane.  The state of a pair is
// 2 D^2 floats (2 or 8 KB): it is read once before the first token and written once after the last.  Serves both
// gka_decode_step (T = 1) and gka_decode_tokens.
#include "gka_common.cuh"

namespace gka {
namespace {

constexpr int kThreadsSmall = 128;     // four pairs per block

template <int D, typename IoT>
__global__ void __launch_bounds__(kThreadsSmall)
decode_small_kernel(float *__restrict__ state, const IoT *__restrict__ q, const IoT *__restrict__ k,
                    const IoT *__restrict__ v, const float *__restrict__ gate, const float *__restrict__ lam,
                    int n_iter, IoT *__restrict__ out, unsigned flags, const float *__restrict__ beta,
                    const float *__restrict__ alpha, int T, int heads, int npairs) {
    const int lane = threadIdx.x & 31;
    const int sh = blockIdx.x * (kThreadsSmall / 32) + (threadIdx.x >> 5);   // (sequence, head) pair of this warp
    if (sh >= npairs) return;
    const int seq = sh / heads, h = sh % heads;
    const bool act = lane < D;                      // lanes from D on carry zeros
    const int row = act ? lane : 0;
    float *gH = state + (size_t)sh * (2 * D * D) + (size_t)row * D;
    float *gU = gH + D * D;

    float Hr[D], Ur[D];
#pragma unroll
    for (int c4 = 0; c4 < D / 4; ++c4) {
        const float4 h4 = act ? *reinterpret_cast<const float4 *>(gH + 4 * c4) : make_float4(0.f, 0.f, 0.f, 0.f);
        const float4 u4 = act ? *reinterpret_cast<const float4 *>(gU + 4 * c4) : make_float4(0.f, 0.f, 0.f, 0.f);
        Hr[4 * c4 + 0] = h4.x; Hr[4 * c4 + 1] = h4.y; Hr[4 * c4 + 2] = h4.z; Hr[4 * c4 + 3] = h4.w;
        Ur[4 * c4 + 0] = u4.x; Ur[4 * c4 + 1] = u4.y; Ur[4 * c4 + 2] = u4.z; Ur[4 * c4 + 3] = u4.w;
    }

    for (int t = 0; t < T; ++t) {
        const size_t tok = ((size_t)seq * T + t) * heads + h;
        // write strength beta (Remark on the beta-augmented variant, Section 4.1): beta k k^T and beta v k^T are the
        // plain writes of sqrt(beta) k and sqrt(beta) v
        const float sb = beta ? sqrtf(fmaxf(beta[tok], 0.f)) : 1.f;
        const float ql = act ? Io<IoT>::load1(q + tok * D + row) : 0.f;
        const float kl = act ? sb * Io<IoT>::load1(k + tok * D + row) : 0.f;
        const float vl = act ? sb * Io<IoT>::load1(v + tok * D + row) : 0.f;
        const float gam = gate[tok];
        float lamv = lam[tok];
        const float al = alpha ? alpha[tok] : 1.f;  // alpha-connection (Section 4.3): the read uses alpha x + (1 - alpha) q

        // ---- H <- gamma H + k k^T, U <- gamma U + v k^T, Frobenius norm of H
        float ss = 0.f;
#pragma unroll
        for (int c = 0; c < D; ++c) {
            const float kc = __shfl_sync(0xffffffffu, kl, c);
            Hr[c] = fmaf(gam, Hr[c], kl * kc);
            Ur[c] = fmaf(gam, Ur[c], vl * kc);
            ss = fmaf(Hr[c], Hr[c], ss);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        const float fro = sqrtf(ss);
        if (flags & GKA_FLAG_ADAPTIVE_LAMBDA) lamv *= fro;

        // ---- Algorithm 1, L = fro + lambda, mu = lambda
        const float Lpm = fro + 2.f * lamv;
        const float rho = fro / Lpm, rho2 = rho * rho, s0 = 2.f / Lpm;
        float omega = 2.f;
        float x = s0 * ql, xp = 0.f;
        for (int it = 0; it < n_iter; ++it) {
            float y = lamv * x;
#pragma unroll
            for (int c = 0; c < D; ++c) y = fmaf(Hr[c], __shfl_sync(0xffffffffu, x, c), y);
            omega = 4.f / (4.f - rho2 * omega);
            const float xn = x - s0 * omega * (y - ql) + (omega - 1.f) * (x - xp);
            xp = x;
            x = xn;
        }

        // ---- read o = U (alpha x + (1 - alpha) q)
        const float xr = alpha ? fmaf(al, x - ql, ql) : x;
        float o = 0.f;
#pragma unroll
        for (int c = 0; c < D; ++c) o = fmaf(Ur[c], __shfl_sync(0xffffffffu, xr, c), o);
        if (act) Io<IoT>::store1(out + tok * D + row, o);
    }

    if (act) {
#pragma unroll
        for (int c4 = 0; c4 < D / 4; ++c4) {
            *reinterpret_cast<float4 *>(gH + 4 * c4) = make_float4(Hr[4 * c4], Hr[4 * c4 + 1], Hr[4 * c4 + 2], Hr[4 * c4 + 3]);
            *reinterpret_cast<float4 *>(gU + 4 * c4) = make_float4(Ur[4 * c4], Ur[4 * c4 + 1], Ur[4 * c4 + 2], Ur[4 * c4 + 3]);
        }
    }
}

template <int D, typename IoT>
cudaError_t launch_small_typed(float *state, const void *q, const void *k, const void *v, const float *gate,
                               const float *lam, int n_iter, void *out, int nseq, int T, int heads, unsigned flags,
                               const float *beta, const float *alpha, cudaEvent_t ev_start, cudaEvent_t ev_stop,
                               cudaStream_t stream) {
    const int npairs = nseq * heads;
    const int blocks = (npairs + kThreadsSmall / 32 - 1) / (kThreadsSmall / 32);
    if (ev_start) cudaEventRecord(ev_start, stream);
    decode_small_kernel<D, IoT><<<blocks, kThreadsSmall, 0, stream>>>(
        state, reinterpret_cast<const IoT *>(q), reinterpret_cast<const IoT *>(k), reinterpret_cast<const IoT *>(v), gate, lam,
        n_iter, reinterpret_cast<IoT *>(out), flags, beta, alpha, T, heads, npairs);
    if (ev_stop) cudaEventRecord(ev_stop, stream);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode_small(float *state, const void *q, const void *k, const void *v, const float *gate,
                                const float *lam, int n_iter, void *out, int nseq, int T, int heads, int d, int io_dtype,
                                unsigned flags, const float *beta, const float *alpha, cudaEvent_t ev_start,
                                cudaEvent_t ev_stop, cudaStream_t stream) {
    if (d == 32)
        return io_dtype == GKA_BF16
                   ? launch_small_typed<32, __nv_bfloat16>(state, q, k, v, gate, lam, n_iter, out, nseq, T, heads, flags, beta, alpha, ev_start, ev_stop, stream)
                   : launch_small_typed<32, float>(state, q, k, v, gate, lam, n_iter, out, nseq, T, heads, flags, beta, alpha, ev_start, ev_stop, stream);
    return io_dtype == GKA_BF16
               ? launch_small_typed<16, __nv_bfloat16>(state, q, k, v, gate, lam, n_iter, out, nseq, T, heads, flags, beta, alpha, ev_start, ev_stop, stream)
               : launch_small_typed<16, float>(state, q, k, v, gate, lam, n_iter, out, nseq, T, heads, flags, beta, alpha, ev_start, ev_stop, stream);
}

}  // namespace gka
