// Shared host/device helpers of the GKA library: work decomposition of the chunked
// forward, workspace layout, I/O type conversion.  No method arithmetic lives here.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/gka.h"

namespace gka {

constexpr int kChunk = 64;            // tokens per chunk (C)
constexpr int kMaxWorkItems = 296;    // upper bound on persistent work items (2 per SM on 148 SMs)
// Division of an index below 2^31 by a divisor fixed for a launch, as a multiplication: with l = ceil(log2 d),
// k = 31 + l and M = floor(2^k / d) + 1, floor(n M / 2^k) = floor(n / d) for every n < 2^31 (the excess
// M d - 2^k is at most d, so the error n (M d - 2^k) / (d 2^k) stays below 1 / d).
struct FastDiv {
    unsigned mul, shift, d;
    __host__ __device__ void set(unsigned div) {
        d = div;
        unsigned l = 0;
        while ((1ull << l) < div) ++l;
        shift = 31 + l;
        mul = (unsigned)((1ull << shift) / div + 1ull);
    }
    __host__ __device__ unsigned div(unsigned n) const { return (unsigned)(((unsigned long long)n * mul) >> shift); }
};

// chunks per sequence: the last one holds the T mod C remaining tokens when T is not a multiple of C
__host__ __device__ constexpr int chunks_of(int T) { return (T + kChunk - 1) / kChunk; }

// ---------------------------------------------------------------------------------------------
// Work decomposition.  The B*heads sequences of N = ceil(T/C) chunks each form one flat list of
// NC = B*heads*N chunks; work item i of G owns the contiguous range [lo(i), lo(i+1)).  A range
// may cover several sequences and may cut a sequence in the middle.  Where an item's range ends
// inside a sequence the item's last run is summarised (decay product, delta-H, delta-U) by the
// summary kernel, the summaries of the items that hold the earlier part of a sequence are folded into
// the start state of the next item (by a scan kernel on the fp32 path, by the main kernel itself on the
// tensor-core path), and the main kernel then processes all items independently, carrying (H, U) on
// chip inside each run.
// Range boundaries are multiples of `unit` chunks: 2 when every sequence has an even number of chunks
// and there are at least two chunks per item (the tensor-core kernel pairs chunks into 128-token tiles;
// even boundaries keep every run an even number of chunks long), else 1.
// ---------------------------------------------------------------------------------------------
struct WorkPlan {
    int BH;        // B * heads
    int N;         // chunks per sequence
    long long NC;  // total chunks
    int G;         // work items
    int unit;      // granularity of the range boundaries in chunks (1 or 2)
    FastDiv divN;  // flat chunk index -> sequence
    __host__ __device__ long long lo(int i) const { return unit * (((long long)i * (NC / unit)) / G); }
    __host__ __device__ void set(int bh, int n, int g, bool pairs = true) {
        BH = bh;
        N = n;
        NC = (long long)bh * n;
        G = g;
        divN.set((unsigned)n);
        unit = (pairs && n % 2 == 0 && 2LL * g <= NC) ? 2 : 1;
    }
    // start of the last run of item i (flat chunk index)
    __host__ __device__ long long last_run_start(int i) const {
        long long l = lo(i), h = lo(i + 1);
        long long s = ((h - 1) / N) * N;
        return s > l ? s : l;
    }
    __host__ __device__ bool cut_out(int i) const { return (lo(i + 1) % N) != 0; }
    __host__ __device__ bool cut_in(int i) const { return (lo(i) % N) != 0; }
};

// Workspace layout (floats): start states [G][st], summaries [G][st], running masters [G][st],
// decay products [G].  st = d_k*d_k + d_v*d_k.
struct Workspace {
    float *start;
    float *delta;
    float *cur;
    float *decay;
};

__host__ __device__ inline size_t state_floats(int dk, int dv) {
    return (size_t)dk * dk + (size_t)dv * dk;
}

inline size_t workspace_bytes_for(int G, int dk, int dv) {
    size_t st = state_floats(dk, dv);
    size_t fl = 3 * (size_t)G * st + (size_t)G;
    return ((fl * sizeof(float) + 255) / 256) * 256;
}

inline Workspace carve_workspace(void *base, int G, int dk, int dv) {
    size_t st = state_floats(dk, dv);
    Workspace w;
    w.start = reinterpret_cast<float *>(base);
    w.delta = w.start + (size_t)G * st;
    w.cur = w.delta + (size_t)G * st;
    w.decay = w.cur + (size_t)G * st;
    return w;
}

// ---------------------------------------------------------------------------------------------
// Tensor-core path (bf16 I/O, d = 128).  Its unit of work is a tile of 128 consecutive tokens of one sequence;
// a sequence is ceil(T / 128) tiles and the WorkPlan above is then a plan over tiles (N = tiles per sequence,
// unit 1).  A state kernel walks the plan's items, carries the fp32 (H, U) on chip and stores, for every tile,
// the bf16 operand copies of the tile-initial H_0 and U_0 and ||H_0||_F^2; the solve kernel then treats the
// tiles as independent problems.  Workspace: start states [G][st], summaries [G][st], decay products [G],
// ||H_0||_F^2 [tiles], bf16 copies [tiles][2][128][128].
// ---------------------------------------------------------------------------------------------
constexpr int kTile = 128;
__host__ __device__ constexpr int tiles_of(int T) { return (T + kTile - 1) / kTile; }
constexpr size_t kTileStateBytes = 2 * 128 * 128 * 2;   // bf16 H_0 and U_0 of one tile

struct TcWorkspace {
    float *start, *delta, *decay, *hh;
    unsigned char *hu;
};
inline size_t tc_workspace_bytes_for(int G, long long ntiles) {
    const size_t st = state_floats(128, 128);
    auto up = [](size_t n) { return (n + 255) / 256 * 256; };
    return 2 * up((size_t)G * st * sizeof(float)) + up((size_t)G * sizeof(float)) + up((size_t)ntiles * sizeof(float)) +
           (size_t)ntiles * kTileStateBytes;
}
inline TcWorkspace carve_tc_workspace(void *base, int G, long long ntiles) {
    const size_t st = state_floats(128, 128);
    auto up = [](size_t n) { return (n + 255) / 256 * 256; };
    unsigned char *p = reinterpret_cast<unsigned char *>(base);
    TcWorkspace w;
    w.start = reinterpret_cast<float *>(p); p += up((size_t)G * st * sizeof(float));
    w.delta = reinterpret_cast<float *>(p); p += up((size_t)G * st * sizeof(float));
    w.decay = reinterpret_cast<float *>(p); p += up((size_t)G * sizeof(float));
    w.hh = reinterpret_cast<float *>(p); p += up((size_t)ntiles * sizeof(float));
    w.hu = p;
    return w;
}

// ---------------------------------------------------------------------------------------------
// I/O element access: T is float or __nv_bfloat16; arithmetic always sees float.
// ---------------------------------------------------------------------------------------------
template <typename T> struct Io;
template <> struct Io<float> {
    static __device__ __forceinline__ float4 load4(const float *p) {
        return *reinterpret_cast<const float4 *>(p);
    }
    static __device__ __forceinline__ void store4(float *p, float4 v) {
        *reinterpret_cast<float4 *>(p) = v;
    }
    static __device__ __forceinline__ float load1(const float *p) { return *p; }
    static __device__ __forceinline__ void store1(float *p, float v) { *p = v; }
};
template <> struct Io<__nv_bfloat16> {
    static __device__ __forceinline__ float4 load4(const __nv_bfloat16 *p) {
        uint2 u = *reinterpret_cast<const uint2 *>(p);
        __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162 *>(&u.x);
        __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162 *>(&u.y);
        float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
        return make_float4(fa.x, fa.y, fb.x, fb.y);
    }
    static __device__ __forceinline__ void store4(__nv_bfloat16 *p, float4 v) {
        __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y);
        __nv_bfloat162 b = __floats2bfloat162_rn(v.z, v.w);
        uint2 u;
        u.x = *reinterpret_cast<uint32_t *>(&a);
        u.y = *reinterpret_cast<uint32_t *>(&b);
        *reinterpret_cast<uint2 *>(p) = u;
    }
    static __device__ __forceinline__ float load1(const __nv_bfloat16 *p) {
        return __bfloat162float(*p);
    }
    static __device__ __forceinline__ void store1(__nv_bfloat16 *p, float v) {
        *p = __float2bfloat16_rn(v);
    }
};

#ifdef __CUDACC__
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

// Wait for an mbarrier phase with a time limit (about a second).  The wait sleeps in hardware
// (try_wait with a suspend-time hint), so a waiting warp leaves the issue slots to working warps.
// Returns false if the phase did not complete in time; the caller records GKA_ERR_TIMEOUT and
// leaves cleanly.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar_addr, uint32_t parity) {
    for (int tries = 0; tries < 200000; ++tries) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar_addr), "r"(parity), "r"(5000u)
            : "memory");
        if (done) return true;
    }
    return false;
}
#endif

// Arguments shared by the chunked-forward kernels.
struct FwdArgs {
    const void *q, *k, *v;
    const float *gate, *lam;
    void *out;
    float *state_out;
    const float *state_in;
    float *fro_out;
    const float *beta;     // optional write strengths [B, T, heads]; nullptr = 1
    const float *alpha;    // optional alpha-connection weights [B, T, heads]; nullptr = 1
    int *device_status;
    int B, T, heads;
    int d;                 // head dimension of the caller's tensors (the tensor path works on 128 channels on chip: 64 is zero-extended)
    FastDiv divH;          // sequence index -> batch entry (divisor: heads)
    int n_iter;
    unsigned flags;
    int after_summary;     // tensor path: the main kernel is launched as a programmatic dependent of the summary kernel
    int start_from_scan;   // tensor path: start states were materialised by the scan kernel (long chains of summaries)
    int state_split;       // tensor path, no sequence cut: two blocks per work item in the state kernel, one for H, one for U
    int solve_only;        // write the solve x_t = CH(H_t + lambda_t I, q_t, r) itself instead of U_t x_t (v unused)
    WorkPlan plan;
    Workspace ws;
    float *tile_hh;        // tensor path: ||H_0||_F^2 of every 128-token tile
    unsigned char *tile_hu; // tensor path: bf16 H_0, U_0 of every 128-token tile
    cudaEvent_t ev_start, ev_stop;   // optional, recorded around the main kernel (host side only)
};

// Launchers implemented in the kernel translation units.  Each returns a cudaError_t.
cudaError_t launch_fwd_simt(const FwdArgs &a, int d, int io_dtype, cudaStream_t stream);
// cross-item scan of the summaries; after_summary: launched as a programmatic dependent of the summary kernel
cudaError_t launch_fwd_scan(const FwdArgs &a, int st, cudaStream_t stream, bool after_summary);
cudaError_t launch_decode(float *state, const void *q, const void *k, const void *v,
                          const float *gate, const float *lam, int n_iter, void *out, int nseq,
                          int heads, int d, int io_dtype, unsigned flags, const float *beta, const float *alpha, int *device_status,
                          cudaEvent_t ev_start, cudaEvent_t ev_stop, cudaStream_t stream);
// head dimensions 16 and 32, T >= 1 tokens per sequence: one warp per (sequence, head) pair
cudaError_t launch_decode_small(float *state, const void *q, const void *k, const void *v, const float *gate,
                                const float *lam, int n_iter, void *out, int nseq, int T, int heads, int d, int io_dtype,
                                unsigned flags, const float *beta, const float *alpha, cudaEvent_t ev_start,
                                cudaEvent_t ev_stop, cudaStream_t stream);
// the same step over T consecutive tokens per sequence, the state read and written once
cudaError_t launch_decode_multi(float *state, const void *q, const void *k, const void *v, const float *gate,
                                const float *lam, int n_iter, void *out, int nseq, int T, int heads, int d, int io_dtype,
                                unsigned flags, const float *beta, const float *alpha, int *device_status,
                                cudaEvent_t ev_start, cudaEvent_t ev_stop, cudaStream_t stream);

}  // namespace gka
