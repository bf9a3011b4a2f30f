// fp32 chunk-wise GKA forward on CUDA cores (sm_100a).
//
// This is the fp32-arithmetic path of gka_fwd_chunked: it serves f32 I/O and GKA_PREC_HIGH.
// It follows the chunk-wise formulation of Section 4.2.1: per chunk of C = 64 tokens, with the
// chunk-initial state (H_0, U_0), cumulative gates zeta and the decay mask
// Gamma[c][j] = zeta_c / zeta_j (j <= c),
//
//     ||H_c||_F    from H_0, K and the Gram matrix K K^T                     (chunk-wise norms)
//     Y = zeta o (X H_0) + (Gamma o (X K^T)) K + lambda o X                  (H_c x_c for all c)
//     Algorithm 1 on all 64 tokens at once, L = ||H_c||_F + lambda_c, mu = lambda_c
//     O = zeta o (X U_0^T) + (Gamma o (X K^T)) V
//     H_C = zeta_C H_0 + K^T diag(Gamma[C]) K,  U_C = zeta_C U_0 + V^T diag(Gamma[C]) K
//
// Three kernels: segment summaries, a scan over segments, and the main kernel (gka_common.cuh
// explains the work decomposition).  One thread block of 256 threads per work item.
#include "gka_common.cuh"

namespace gka {
namespace {

constexpr int kThreads = 256;
constexpr int XS = 68;  // padded stride (floats) of tiles stored [channel][token]

template <int D> struct Cfg {
    static constexpr int DG = D / 64;   // float4 groups per thread along channels
    static constexpr int NCH = 4 * DG;  // channels per thread
    static constexpr int kSmemFloats = D * D + 2 * D * XS + 2 * kChunk * D + kChunk * XS + 8 * kChunk + 64;
    static constexpr size_t kSmemBytes = (size_t)kSmemFloats * sizeof(float);
};

__device__ __forceinline__ float4 ld4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ void st4(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }

// acc[t][g*4+u] += sum_kk At[kk][4tc+t] * Bm[kk][64g + 4td + u]
template <int D>
__device__ __forceinline__ void gemm_tok_mat(float (&acc)[4][Cfg<D>::NCH], const float *At,
                                             const float *Bm, int Kdim, int tc, int td) {
#pragma unroll 4
    for (int kk = 0; kk < Kdim; ++kk) {
        float4 xv = ld4(At + kk * XS + 4 * tc);
        float xa[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
        for (int g = 0; g < Cfg<D>::DG; ++g) {
            float4 hv = ld4(Bm + kk * D + 64 * g + 4 * td);
            float ha[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
                for (int u = 0; u < 4; ++u) acc[t][4 * g + u] = fmaf(xa[t], ha[u], acc[t][4 * g + u]);
        }
    }
}

// s[t][u] = sum_d At[d][4tc+t] * Bt[d][4td+u]
template <int D>
__device__ __forceinline__ void gemm_tok_tok(float (&s)[4][4], const float *At, const float *Bt,
                                             int tc, int td) {
#pragma unroll
    for (int t = 0; t < 4; ++t)
#pragma unroll
        for (int u = 0; u < 4; ++u) s[t][u] = 0.f;
#pragma unroll 4
    for (int d = 0; d < D; ++d) {
        float4 xv = ld4(At + d * XS + 4 * tc);
        float4 kv = ld4(Bt + d * XS + 4 * td);
        float xa[4] = {xv.x, xv.y, xv.z, xv.w};
        float ka[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
        for (int t = 0; t < 4; ++t)
#pragma unroll
            for (int u = 0; u < 4; ++u) s[t][u] = fmaf(xa[t], ka[u], s[t][u]);
    }
}

// M (global, [D][D]) <- zetaC * M + sum_j A[j][row] * w[j] * K[j][col];  A, K: smem [64][D].
template <int D>
__device__ __forceinline__ void state_update(float *M, const float *A, const float *K, const float *w,
                                             float zetaC, bool first_is_zero) {
    constexpr int DG = Cfg<D>::DG, NCH = Cfg<D>::NCH;
    const int tr = threadIdx.x >> 4, tcn = threadIdx.x & 15;
    float acc[NCH][NCH];
#pragma unroll
    for (int i = 0; i < NCH; ++i)
#pragma unroll
        for (int j = 0; j < NCH; ++j) acc[i][j] = 0.f;
#pragma unroll 2
    for (int j = 0; j < kChunk; ++j) {
        const float wj = w[j];
        float ar[NCH], kc[NCH];
#pragma unroll
        for (int g = 0; g < DG; ++g) {
            float4 a4 = ld4(A + j * D + 64 * g + 4 * tr);
            float4 k4 = ld4(K + j * D + 64 * g + 4 * tcn);
            ar[4 * g + 0] = a4.x * wj; ar[4 * g + 1] = a4.y * wj;
            ar[4 * g + 2] = a4.z * wj; ar[4 * g + 3] = a4.w * wj;
            kc[4 * g + 0] = k4.x; kc[4 * g + 1] = k4.y; kc[4 * g + 2] = k4.z; kc[4 * g + 3] = k4.w;
        }
#pragma unroll
        for (int i = 0; i < NCH; ++i)
#pragma unroll
            for (int c = 0; c < NCH; ++c) acc[i][c] = fmaf(ar[i], kc[c], acc[i][c]);
    }
#pragma unroll
    for (int gi = 0; gi < DG; ++gi)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = 64 * gi + 4 * tr + i;
#pragma unroll
            for (int gc = 0; gc < DG; ++gc) {
                float *p = M + (size_t)row * D + 64 * gc + 4 * tcn;
                float4 o = first_is_zero ? make_float4(0.f, 0.f, 0.f, 0.f) : ld4(p);
                o.x = fmaf(zetaC, o.x, acc[4 * gi + i][4 * gc + 0]);
                o.y = fmaf(zetaC, o.y, acc[4 * gi + i][4 * gc + 1]);
                o.z = fmaf(zetaC, o.z, acc[4 * gi + i][4 * gc + 2]);
                o.w = fmaf(zetaC, o.w, acc[4 * gi + i][4 * gc + 3]);
                st4(p, o);
            }
        }
}

// Load one chunk's rows of a [B,T,heads,D] tensor into smem row-major (dst) and, optionally,
// transposed with stride XS (dstT[d][token]).  With write strengths (beta-augmented variant, Remark in
// Section 4.1) key and value rows are scaled by sqrt(beta_t): beta k k^T and beta v k^T are the plain writes of
// the scaled rows, and every later use of a key in the chunk-wise form carries exactly this factor.
// Rows from nvalid on (the last chunk of a sequence whose length is not a multiple of C) are zero: a zero key
// and value write nothing, a zero query solves to zero.  The caller's rows hold dx <= D channels (head dimensions 16
// and 32 run on the 64-channel kernels, zero-extended: zero channels write nothing and solve to zero).
template <int D, typename IoT>
__device__ __forceinline__ void load_rows(const IoT *src, size_t row0_elem, size_t row_stride_elem,
                                          float *dst, float *dstT, int nvalid, int dx, const float *beta = nullptr,
                                          size_t tok0 = 0, int heads = 0) {
    constexpr int F4 = D / 4;
    for (int idx = threadIdx.x; idx < kChunk * F4; idx += kThreads) {
        const int row = idx / F4, c4 = idx % F4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);      // channels from dx on (a smaller head dimension, zero-extended) are zero
        if (row < nvalid && 4 * c4 < dx) v = Io<IoT>::load4(src + row0_elem + (size_t)row * row_stride_elem + 4 * c4);
        if (beta && row < nvalid) {
            const float sb = sqrtf(fmaxf(beta[tok0 + (size_t)row * heads], 0.f));
            v.x *= sb; v.y *= sb; v.z *= sb; v.w *= sb;
        }
        if (dst) st4(dst + row * D + 4 * c4, v);
        if (dstT) {
            dstT[(4 * c4 + 0) * XS + row] = v.x;
            dstT[(4 * c4 + 1) * XS + row] = v.y;
            dstT[(4 * c4 + 2) * XS + row] = v.z;
            dstT[(4 * c4 + 3) * XS + row] = v.w;
        }
    }
}

__device__ __forceinline__ float block_sum(float v, float *red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i) t += red[i];
    return t;
}

// Gates of one chunk: G[c] = sum_{i<=c} log gamma_i (clamped), zeta = exp(G), w[j] = exp(G[C-1]-G[j]).
__device__ __forceinline__ void load_gates(const float *gate, const float *lam, size_t tok0, int heads, int nvalid,
                                           float *sG, float *sZeta, float *sLam, float *sW) {
    const int c = threadIdx.x;
    if (c < kChunk) {      // past the sequence: no decay, any positive lambda
        sW[c] = c < nvalid ? fmaxf(logf(gate[tok0 + (size_t)c * heads]), -80.f) : 0.f;  // temporary: log gamma
        sLam[c] = c < nvalid ? lam[tok0 + (size_t)c * heads] : 1.f;
    }
    __syncthreads();
    float g = 0.f;
    if (c < kChunk) {
        for (int i = 0; i <= c; ++i) g += sW[i];
    }
    __syncthreads();
    if (c < kChunk) {
        sG[c] = g;
        sZeta[c] = expf(g);
    }
    __syncthreads();
    if (c < kChunk) sW[c] = expf(sG[kChunk - 1] - sG[c]);
    __syncthreads();
}

// ------------------------------------------------------------------------------------------
// Segment summaries: for every work item whose range ends inside a sequence, the decay product
// and the (delta-H, delta-U) of its last run, relative to a zero start state.
// ------------------------------------------------------------------------------------------
template <int D, typename IoT>
__global__ void __launch_bounds__(kThreads, 1) fwd_simt_summary(FwdArgs a) {
    extern __shared__ __align__(16) float smem[];
    const WorkPlan &P = a.plan;
    const int item = blockIdx.x;
    if (!P.cut_out(item)) return;
    float *sK = smem;
    float *sV = sK + kChunk * D;
    float *sG = sV + kChunk * D;
    float *sZeta = sG + kChunk, *sLam = sZeta + kChunk, *sW = sLam + kChunk;
    const size_t st = state_floats(D, D);
    float *dH = a.ws.delta + (size_t)item * st;
    float *dU = dH + (size_t)D * D;
    const long long f0 = P.last_run_start(item), f1 = P.lo(item + 1);
    const int seq = (int)(f0 / P.N), b = seq / a.heads, h = seq % a.heads;
    const size_t rs = (size_t)a.heads * a.d;
    float decay_log = 0.f;
    for (long long f = f0; f < f1; ++f) {
        const int n = (int)(f % P.N);
        const size_t tok0 = ((size_t)b * a.T + (size_t)n * kChunk) * a.heads + h;
        const int nvalid = min(kChunk, a.T - n * kChunk);
        load_rows<D, IoT>(reinterpret_cast<const IoT *>(a.k), tok0 * a.d, rs, sK, nullptr, nvalid, a.d, a.beta, tok0, a.heads);
        load_rows<D, IoT>(reinterpret_cast<const IoT *>(a.v), tok0 * a.d, rs, sV, nullptr, nvalid, a.d, a.beta, tok0, a.heads);
        load_gates(a.gate, a.lam, tok0, a.heads, nvalid, sG, sZeta, sLam, sW);
        const float zc = sZeta[kChunk - 1];
        decay_log += sG[kChunk - 1];
        state_update<D>(dH, sK, sK, sW, zc, f == f0);
        state_update<D>(dU, sV, sK, sW, zc, f == f0);
        __syncthreads();
    }
    if (threadIdx.x == 0) a.ws.decay[item] = expf(decay_log);
}

// ------------------------------------------------------------------------------------------
// Scan over work items: the start state of item i (when its range starts inside a sequence) is the
// fold  state <- decay_j * state + delta_j  over the items j < i that hold the earlier part of the
// same sequence, starting from the sequence's initial state.  A sequence spans few items, so every
// item folds its own short chain independently: blockIdx.y = item, four state elements per thread.
// ------------------------------------------------------------------------------------------
__global__ void fwd_scan(FwdArgs a, int st) {
    // On the tensor-core path this kernel is a programmatic dependent of the summary kernel and the main kernel one of
    // this kernel: both may be scheduled early, and each waits here for its producer (no effect on plain launches).
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const WorkPlan &P = a.plan;
    const int i = blockIdx.y + 1;
    __shared__ int s_j0, s_seq;           // the chain is found once per block (64-bit divisions are slow)
    if (threadIdx.x == 0) {
        int j0 = -1;
        if (P.cut_in(i)) {
            // first item of the chain: the one whose range holds the start of this sequence (its last run
            // begins there, whatever sequence the item itself started in)
            const long long seq_start = (P.lo(i) / P.N) * P.N;
            j0 = i - 1;
            while (P.lo(j0) > seq_start) --j0;
        }
        s_j0 = j0;
        s_seq = (int)(P.lo(i) / P.N);
    }
    __syncthreads();
    const int j0 = s_j0, seq = s_seq;
    if (j0 < 0) return;
    const int e = 4 * (blockIdx.x * blockDim.x + threadIdx.x);
    if (e >= st) return;
    float4 carry = make_float4(0.f, 0.f, 0.f, 0.f);
    if (a.state_in) {
        const int dd = 2 * a.d * a.d;
        if (dd == st) {
            carry = ld4(a.state_in + (size_t)seq * st + e);
        } else {
            // the workspace holds states zero-extended to the on-chip head dimension (128 or 64)
            const int Dw = st == 2 * 128 * 128 ? 128 : 64;
            const int which = e / (Dw * Dw), row = (e / Dw) % Dw, col = e % Dw;
            if (row < a.d && col < a.d) carry = ld4(a.state_in + (size_t)seq * dd + (size_t)which * a.d * a.d + (size_t)row * a.d + col);
        }
    }
    for (int j = j0; j < i; ++j) {
        const float dcy = a.ws.decay[j];
        const float4 d = ld4(a.ws.delta + (size_t)j * st + e);
        carry.x = fmaf(dcy, carry.x, d.x);
        carry.y = fmaf(dcy, carry.y, d.y);
        carry.z = fmaf(dcy, carry.z, d.z);
        carry.w = fmaf(dcy, carry.w, d.w);
    }
    st4(a.ws.start + (size_t)i * st + e, carry);
}

// ------------------------------------------------------------------------------------------
// Main kernel.
// ------------------------------------------------------------------------------------------
template <int D, typename IoT>
__global__ void __launch_bounds__(kThreads, 1) fwd_simt_main(FwdArgs a) {
    constexpr int DG = Cfg<D>::DG, NCH = Cfg<D>::NCH;
    extern __shared__ __align__(16) float smem[];
    float *sH = smem;                      // [D][D]  H_0, later U_0^T
    float *sXt = sH + D * D;               // [D][XS] X^T
    float *sKt = sXt + D * XS;             // [D][XS] K^T
    float *sK = sKt + D * XS;              // [64][D]
    float *sV = sK + kChunk * D;           // [64][D]
    float *sPt = sV + kChunk * D;          // [64][XS] P^T: sPt[j][c]
    float *sG = sPt + kChunk * XS;
    float *sZeta = sG + kChunk, *sLam = sZeta + kChunk, *sW = sLam + kChunk;
    float *sF = sW + kChunk, *sA = sF + kChunk, *sDj = sA + kChunk, *sTmp = sDj + kChunk;
    float *sRed = sTmp + kChunk;

    const WorkPlan &P = a.plan;
    const int item = blockIdx.x;
    const int tid = threadIdx.x, tc = tid >> 4, td = tid & 15;
    const size_t st = state_floats(D, D);
    float *mH = a.ws.cur + (size_t)item * st;   // running masters of this work item
    float *mU = mH + (size_t)D * D;
    const IoT *gq = reinterpret_cast<const IoT *>(a.q);
    IoT *gout = reinterpret_cast<IoT *>(a.out);
    const size_t rs = (size_t)a.heads * a.d;
    const int dx = a.d;                         // channels of the caller's rows and states (dx <= D)
    const size_t ste = 2 * (size_t)dx * dx;
    const bool adaptive = (a.flags & GKA_FLAG_ADAPTIVE_LAMBDA) != 0;

    const long long f_lo = P.lo(item), f_hi = P.lo(item + 1);
    for (long long f = f_lo; f < f_hi; ++f) {
        const int seq = (int)(f / P.N), n = (int)(f % P.N);
        const int b = seq / a.heads, h = seq % a.heads;
        const size_t tok0 = ((size_t)b * a.T + (size_t)n * kChunk) * a.heads + h;
        const int nvalid = min(kChunk, a.T - n * kChunk);     // tokens of this chunk that exist

        // ---- run start: fetch the start state into the running masters
        if (f == f_lo || n == 0) {
            if (n != 0 || dx == D) {
                const float *src = (n == 0) ? (a.state_in ? a.state_in + (size_t)seq * st : nullptr)
                                            : a.ws.start + (size_t)item * st;
                for (size_t e = 4 * (size_t)tid; e < st; e += 4 * kThreads)
                    st4(mH + e, src ? ld4(src + e) : make_float4(0.f, 0.f, 0.f, 0.f));
            } else {
                // the caller's state has dx x dx matrices: zero-extended to D x D
                const float *src = a.state_in ? a.state_in + (size_t)seq * ste : nullptr;
                for (size_t e = 4 * (size_t)tid; e < st; e += 4 * kThreads) {
                    const int which = (int)(e / (D * D)), row = (int)(e / D) % D, col = (int)(e % D);
                    const bool in = src && row < dx && col < dx;
                    st4(mH + e, in ? ld4(src + (size_t)which * dx * dx + (size_t)row * dx + col) : make_float4(0.f, 0.f, 0.f, 0.f));
                }
            }
        }
        __syncthreads();

        // ---- stage the chunk
        load_rows<D, IoT>(reinterpret_cast<const IoT *>(a.k), tok0 * dx, rs, sK, sKt, nvalid, dx, a.beta, tok0, a.heads);
        load_rows<D, IoT>(reinterpret_cast<const IoT *>(a.v), tok0 * dx, rs, sV, nullptr, nvalid, dx, a.beta, tok0, a.heads);
        for (int e = 4 * tid; e < D * D; e += 4 * kThreads) st4(sH + e, ld4(mH + e));
        load_gates(a.gate, a.lam, tok0, a.heads, nvalid, sG, sZeta, sLam, sW);  // ends with a barrier

        // ---- chunk-wise Frobenius norms (Section 4.2.1), O(C^2) form:
        //      f_c^2 = zeta_c^2 ||H_0||^2 + sum_{j<=c} Gamma[c][j]^2 d_j,
        //      d_j   = 2 zeta_j k_j^T H_0 k_j + 2 sum_{i<j} Gamma[j][i] (k_j.k_i)^2 + (k_j.k_j)^2
        float hh = 0.f;
        for (int e = 4 * tid; e < D * D; e += 4 * kThreads) {
            float4 v4 = ld4(sH + e);
            hh += v4.x * v4.x + v4.y * v4.y + v4.z * v4.z + v4.w * v4.w;
        }
        hh = block_sum(hh, sRed);
        {
            float acc[4][NCH];
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
                for (int u = 0; u < NCH; ++u) acc[t][u] = 0.f;
            gemm_tok_mat<D>(acc, sKt, sH, D, tc, td);   // (K H_0)[j][d]
            float part[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                float s = 0.f;
#pragma unroll
                for (int g = 0; g < DG; ++g) {
                    float4 kv = ld4(sK + (4 * tc + t) * D + 64 * g + 4 * td);
                    s += acc[t][4 * g + 0] * kv.x + acc[t][4 * g + 1] * kv.y +
                         acc[t][4 * g + 2] * kv.z + acc[t][4 * g + 3] * kv.w;
                }
                part[t] = s;
            }
            float gm[4][4];
            gemm_tok_tok<D>(gm, sKt, sKt, tc, td);      // Gram[j][i], j = 4tc+t, i = 4td+u
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int j = 4 * tc + t;
                float s = 2.f * sZeta[j] * part[t];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = 4 * td + u;
                    const float g2 = gm[t][u] * gm[t][u];
                    if (i < j) s += 2.f * expf(sG[j] - sG[i]) * g2;
                    else if (i == j) s += g2;
                }
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                if (td == 0) sDj[j] = s;
            }
        }
        __syncthreads();
        if (tid < kChunk) {
            const int c = tid;
            float s = sZeta[c] * sZeta[c] * hh;
            for (int j = 0; j <= c; ++j) s += expf(2.f * (sG[c] - sG[j])) * sDj[j];
            const float fc = sqrtf(fmaxf(s, 0.f));
            sF[c] = fc;
            if (adaptive) sLam[c] = sLam[c] * fc;
            if (a.fro_out && c < nvalid) a.fro_out[tok0 + (size_t)c * a.heads] = fc;
        }
        __syncthreads();

        // ---- Algorithm 1 on the whole chunk, in residual form: with d_i = x_i - x_{i-1} (x_{-1} = 0, d_0 = x_0) the update
        // x_{i+1} = x_i + (omega - 1) d_i + (2 omega / (L + mu)) (q - A x_i) reads r_i = r_{i-1} - A d_i (r_{-1} = q),
        // d_{i+1} = (omega - 1) d_i + (2 omega / (L + mu)) r_i, x_{i+1} = x_i + d_{i+1}: the same iterates in exact
        // arithmetic, but the matrix meets the shrinking increment, so its rounding errors shrink with it.
        // xm: iterate x; xp: increment d (the published operand); qm: q - (A - lambda) x (the lambda term uses x itself)
        float xm[4][NCH], xp[4][NCH], qm[4][NCH];
        float omega[4], rho2[4], s0[4], lamr[4], zet[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int c = 4 * tc + t;
            const float fc = sF[c], lc = sLam[c];
            const float Lpm = fc + 2.f * lc;            // L + mu
            const float rho = fc / Lpm;                 // (L - mu) / (L + mu)
            rho2[t] = rho * rho;
            s0[t] = 2.f / Lpm;
            lamr[t] = lc;
            zet[t] = sZeta[c];
            omega[t] = 2.f;
#pragma unroll
            for (int g = 0; g < DG; ++g) {
                float4 qv = make_float4(0.f, 0.f, 0.f, 0.f);
                if (c < nvalid && 64 * g + 4 * td < dx) qv = Io<IoT>::load4(gq + (tok0 + (size_t)c * a.heads) * dx + 64 * g + 4 * td);
                qm[t][4 * g + 0] = qv.x; qm[t][4 * g + 1] = qv.y;
                qm[t][4 * g + 2] = qv.z; qm[t][4 * g + 3] = qv.w;
            }
#pragma unroll
            for (int u = 0; u < NCH; ++u) {
                xp[t][u] = s0[t] * qm[t][u];            // d_0 = xi_0 = 2 q / (L + mu)
                xm[t][u] = 0.f;                         // xi_{-1} = 0
            }
        }
        auto publish = [&](const float(&x)[4][NCH]) {
#pragma unroll
            for (int g = 0; g < DG; ++g)
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    st4(sXt + (64 * g + 4 * td + u) * XS + 4 * tc,
                        make_float4(x[0][4 * g + u], x[1][4 * g + u], x[2][4 * g + u], x[3][4 * g + u]));
        };
        auto publish_x = [&]() { publish(xm); };
        auto masked_scores = [&]() {   // sPt[j][c] = Gamma[c][j] * (x_c . k_j), j <= c
            float s[4][4];
            gemm_tok_tok<D>(s, sXt, sKt, tc, td);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int j = 4 * td + u;
                float p[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int c = 4 * tc + t;
                    p[t] = (j <= c) ? expf(sG[c] - sG[j]) * s[t][u] : 0.f;
                }
                st4(sPt + j * XS + 4 * tc, make_float4(p[0], p[1], p[2], p[3]));
            }
        };
        publish(xp);
        __syncthreads();
        for (int it = 0; it < a.n_iter; ++it) {
            masked_scores();                                   // of the increment
            __syncthreads();
            float acc[4][NCH];
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
                for (int u = 0; u < NCH; ++u) acc[t][u] = 0.f;
            gemm_tok_mat<D>(acc, sXt, sH, D, tc, td);          // D H_0
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
                for (int u = 0; u < NCH; ++u) acc[t][u] *= zet[t];
            gemm_tok_mat<D>(acc, sPt, sK, kChunk, tc, td);     // + P K
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                omega[t] = 4.f / (4.f - rho2[t] * omega[t]);   // weight schedule
                const float step = s0[t] * omega[t];
                const float mom = omega[t] - 1.f;
#pragma unroll
                for (int u = 0; u < NCH; ++u) {
                    xm[t][u] += xp[t][u];                                      // x_i
                    qm[t][u] -= acc[t][u];                                     // q - H_c x_i
                    const float res = fmaf(-lamr[t], xm[t][u], qm[t][u]);      // r_i = q - (H_c + lambda_c I) x_i
                    xp[t][u] = fmaf(step, res, mom * xp[t][u]);                // d_{i+1}
                }
            }
            __syncthreads();      // every read of sXt / sPt of this iteration is done
            publish(xp);
            __syncthreads();
        }
#pragma unroll
        for (int t = 0; t < 4; ++t)
#pragma unroll
            for (int u = 0; u < NCH; ++u) xm[t][u] += xp[t][u];               // the final iterate
        if (!a.solve_only && !a.alpha) {
            publish_x();
            __syncthreads();
        }

        if (a.solve_only) {      // the solve itself is the result (Section 4.2.2, Lemma 2: the same solve gives dq from dx)
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int c = 4 * tc + t;
#pragma unroll
                for (int g = 0; g < DG && c < nvalid; ++g)
                    if (64 * g + 4 * td < dx)
                    Io<IoT>::store4(gout + (tok0 + (size_t)c * a.heads) * dx + 64 * g + 4 * td,
                                    make_float4(xm[t][4 * g + 0], xm[t][4 * g + 1], xm[t][4 * g + 2], xm[t][4 * g + 3]));
            }
        }
        if (a.alpha && !a.solve_only) {    // alpha-connection (Section 4.3): the read uses alpha x + (1 - alpha) q
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int c = 4 * tc + t;
                const float al = (c < nvalid) ? a.alpha[tok0 + (size_t)c * a.heads] : 1.f;
#pragma unroll
                for (int g = 0; g < DG; ++g) {      // the query again (its registers hold the residual)
                    float4 qv = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (c < nvalid && 64 * g + 4 * td < dx) qv = Io<IoT>::load4(gq + (tok0 + (size_t)c * a.heads) * dx + 64 * g + 4 * td);
                    xm[t][4 * g + 0] = fmaf(al, xm[t][4 * g + 0] - qv.x, qv.x);
                    xm[t][4 * g + 1] = fmaf(al, xm[t][4 * g + 1] - qv.y, qv.y);
                    xm[t][4 * g + 2] = fmaf(al, xm[t][4 * g + 2] - qv.z, qv.z);
                    xm[t][4 * g + 3] = fmaf(al, xm[t][4 * g + 3] - qv.w, qv.w);
                }
            }
            publish_x();
            __syncthreads();
        }
        // ---- output O = zeta o (X U_0^T) + P V
        masked_scores();
        for (int idx = tid; idx < D * (D / 4); idx += kThreads) {   // sH <- U_0^T
            const int i = idx / (D / 4), e4 = idx % (D / 4);
            float4 uv = ld4(mU + (size_t)i * D + 4 * e4);
            sH[(4 * e4 + 0) * D + i] = uv.x;
            sH[(4 * e4 + 1) * D + i] = uv.y;
            sH[(4 * e4 + 2) * D + i] = uv.z;
            sH[(4 * e4 + 3) * D + i] = uv.w;
        }
        __syncthreads();
        {
            float acc[4][NCH];
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
                for (int u = 0; u < NCH; ++u) acc[t][u] = 0.f;
            gemm_tok_mat<D>(acc, sXt, sH, D, tc, td);
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
                for (int u = 0; u < NCH; ++u) acc[t][u] *= zet[t];
            gemm_tok_mat<D>(acc, sPt, sV, kChunk, tc, td);
#pragma unroll
            for (int t = 0; t < 4 && !a.solve_only; ++t) {
                const int c = 4 * tc + t;
#pragma unroll
                for (int g = 0; g < DG && c < nvalid; ++g)
                    if (64 * g + 4 * td < dx)
                    Io<IoT>::store4(gout + (tok0 + (size_t)c * a.heads) * dx + 64 * g + 4 * td,
                                    make_float4(acc[t][4 * g + 0], acc[t][4 * g + 1],
                                                acc[t][4 * g + 2], acc[t][4 * g + 3]));
            }
        }

        // ---- state carry
        const float zc = sZeta[kChunk - 1];
        state_update<D>(mH, sK, sK, sW, zc, false);
        state_update<D>(mU, sV, sK, sW, zc, false);
        __syncthreads();
        if (n == P.N - 1 && a.state_out) {
            if (dx == D) {
                float *dst = a.state_out + (size_t)seq * st;
                for (size_t e = 4 * (size_t)tid; e < st; e += 4 * kThreads) st4(dst + e, ld4(mH + e));
            } else {                                   // the caller's dx x dx matrices out of the D x D masters
                float *dst = a.state_out + (size_t)seq * ste;
                for (size_t e = 4 * (size_t)tid; e < st; e += 4 * kThreads) {
                    const int which = (int)(e / (D * D)), row = (int)(e / D) % D, col = (int)(e % D);
                    if (row < dx && col < dx) st4(dst + (size_t)which * dx * dx + (size_t)row * dx + col, ld4(mH + e));
                }
            }
        }
        __syncthreads();
    }
}

// Summary + scan pass (only when some work item starts inside a sequence).
template <int D, typename IoT>
cudaError_t launch_summary_scan_typed(const FwdArgs &a, cudaStream_t stream) {
    const int G = a.plan.G;
    const int st = (int)state_floats(D, D);
    bool any_cut = false;
    for (int i = 0; i + 1 < G; ++i) any_cut |= a.plan.cut_out(i);
    if (!any_cut) return cudaSuccess;
    const size_t sm_sum = (size_t)(2 * kChunk * D + 4 * kChunk) * sizeof(float);
    cudaError_t err = cudaFuncSetAttribute(fwd_simt_summary<D, IoT>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_sum);
    if (err != cudaSuccess) return err;
    fwd_simt_summary<D, IoT><<<G, kThreads, sm_sum, stream>>>(a);
    if (G > 1) fwd_scan<<<dim3((st / 4 + 255) / 256, G - 1), 256, 0, stream>>>(a, st);
    return cudaGetLastError();
}

template <int D, typename IoT>
cudaError_t launch_typed(const FwdArgs &a, cudaStream_t stream) {
    cudaError_t err = launch_summary_scan_typed<D, IoT>(a, stream);
    if (err != cudaSuccess) return err;
    err = cudaFuncSetAttribute(fwd_simt_main<D, IoT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)Cfg<D>::kSmemBytes);
    if (err != cudaSuccess) return err;
    if (a.ev_start) cudaEventRecord(a.ev_start, stream);
    fwd_simt_main<D, IoT><<<a.plan.G, kThreads, Cfg<D>::kSmemBytes, stream>>>(a);
    if (a.ev_stop) cudaEventRecord(a.ev_stop, stream);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fwd_scan(const FwdArgs &a, int st, cudaStream_t stream, bool after_summary) {
    if (a.plan.G <= 1) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((st / 4 + 255) / 256, a.plan.G - 1);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = after_summary ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, fwd_scan, a, st);
}

cudaError_t launch_fwd_simt(const FwdArgs &a, int d, int io_dtype, cudaStream_t stream) {
    // head dimensions 16, 32 and 64 run on the 64-channel kernels (a.d is the caller's head dimension)
    if (d == 128) {
        return io_dtype == GKA_BF16 ? launch_typed<128, __nv_bfloat16>(a, stream)
                                    : launch_typed<128, float>(a, stream);
    }
    return io_dtype == GKA_BF16 ? launch_typed<64, __nv_bfloat16>(a, stream)
                                : launch_typed<64, float>(a, stream);
}

}  // namespace gka
