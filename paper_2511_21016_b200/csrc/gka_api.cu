// C ABI of the GKA library: argument validation, work planning and kernel dispatch.
// Every step of the path runs in the kernels of this library; nothing here computes.
#include <stdio.h>

#include <mutex>
#include <vector>

#include "gka_common.cuh"

namespace gka {

cudaError_t launch_fwd_tc(const FwdArgs &a, cudaStream_t stream);   // gka_tc.cu
bool fwd_tc_available();

namespace {

constexpr int kMaxDevices = 64;
int g_sm_count[kMaxDevices] = {};      // per device ordinal; filled on first use (a benign race: every writer stores the same value)
thread_local char g_detail[256] = "";

gka_status cuda_result(cudaError_t err, const char *where) {
    if (err == cudaSuccess) return GKA_OK;
    snprintf(g_detail, sizeof(g_detail), "%s: %s (%s)", where, cudaGetErrorName(err), cudaGetErrorString(err));
    (void)cudaGetLastError();   // clear the sticky launch error so that later calls are not poisoned
    return GKA_ERR_CUDA;
}

int sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return -1;
    if (dev >= 0 && dev < kMaxDevices && g_sm_count[dev] > 0) return g_sm_count[dev];
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
    if (dev >= 0 && dev < kMaxDevices) g_sm_count[dev] = n;
    return n;
}

// Domain check of the per-token scalars (GKA_FLAG_VALIDATE): gamma_t in (0, 1] (Section 4.1, "Adaptive Weighting"),
// lambda_t > 0, or a > 0 with the adaptive rule, so that L >= mu > 0 (the input condition of Algorithm 1), beta_t >= 0,
// all finite.  One pass; the first violation stores GKA_ERR_DOMAIN.
__global__ void validate_kernel(const float *gate, const float *lam, const float *beta, const float *alpha, size_t n,
                                int *device_status) {
    bool bad = false;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float g = gate[i], l = lam[i];
        bad |= !(g > 0.f && g <= 1.f) || !(l > 0.f && l < INFINITY);
        if (beta) bad |= !(beta[i] >= 0.f && beta[i] < INFINITY);
        if (alpha) bad |= !(fabsf(alpha[i]) < INFINITY);
    }
    if (__syncthreads_or(bad) && threadIdx.x == 0) atomicCAS(device_status, (int)GKA_OK, (int)GKA_ERR_DOMAIN);
}
cudaError_t launch_validate(const gka_desc *d, const float *gate, const float *lam, size_t n, cudaStream_t stream) {
    if (!(d->flags & GKA_FLAG_VALIDATE) || !d->device_status) return cudaSuccess;
    const int blocks = (int)((n + 255) / 256 < 592 ? (n + 255) / 256 : 592);
    validate_kernel<<<blocks, 256, 0, stream>>>(gate, lam, d->beta, d->alpha, n, d->device_status);
    return cudaGetLastError();
}

// Self-test of the bounded waits: one block waits, with a limit of a few thousand polls, on an mbarrier that nothing
// arrives at (no copy and no product is outstanding), stores GKA_ERR_TIMEOUT and returns.
__global__ void bounded_wait_selftest_kernel(int polls, int *device_status) {
    __shared__ __align__(8) uint64_t bar;
    const uint32_t addr = smem_u32(&bar);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(addr));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool done = false;
    for (int i = 0; i < polls && !done; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(addr), "r"(0u)
            : "memory");
        done = ok != 0;
    }
    if (__syncthreads_or(!done) && threadIdx.x == 0 && device_status) atomicExch(device_status, (int)GKA_ERR_TIMEOUT);
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned4(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

gka_status check_desc_common(const gka_desc *d) {
    if (!d) return GKA_ERR_NULL;
    if (d->B <= 0 || d->heads <= 0 || d->d_k <= 0 || d->d_v <= 0) return GKA_ERR_SHAPE;
    if (d->d_k != d->d_v) return GKA_ERR_SHAPE;
    if (d->io_dtype != GKA_F32 && d->io_dtype != GKA_BF16) return GKA_ERR_DTYPE;
    if (d->precision != GKA_PREC_NATIVE && d->precision != GKA_PREC_HIGH) return GKA_ERR_DTYPE;
    if (d->d_k != 16 && d->d_k != 32 && d->d_k != 64 && d->d_k != 128) return GKA_ERR_UNSUPPORTED;
    if (d->flags & ~(unsigned)(GKA_FLAG_ADAPTIVE_LAMBDA | GKA_FLAG_VALIDATE)) return GKA_ERR_UNSUPPORTED;
    return GKA_OK;
}

gka_status check_fwd_shape(const gka_desc *d, int chunk) {
    gka_status s = check_desc_common(d);
    if (s != GKA_OK) return s;
    if (chunk != kChunk) return chunk <= 0 ? GKA_ERR_SHAPE : GKA_ERR_UNSUPPORTED;
    if (d->T <= 0) return GKA_ERR_SHAPE;
    if ((long long)d->B * d->heads * chunks_of(d->T) >= (1LL << 31)) return GKA_ERR_UNSUPPORTED;   // 32-bit chunk indices
    return GKA_OK;
}

// bf16 I/O with bf16 tensor-core operands: the tcgen05 kernels, which work on 128-token tiles of 128 channels (head
// dimension 64 is zero-extended on chip: the loads of the upper 64 channels read past the tensor, i.e. zeros)
// Sequences of fewer than 16 tokens stay on the fp32 kernels: right after a zero initial state H_t is all but rank one,
// x_t is dominated by q_t / lambda_t off the key direction while the read takes only its key component, and bf16
// operands resolve that component to a few percent (up to 16 % for one token under the adaptive rule); from about a
// dozen tokens on such tokens are a negligible part of the output.
constexpr int kMinTensorT = 16;
bool wants_tensor_path(const gka_desc *d) {
    return d->io_dtype == GKA_BF16 && d->precision == GKA_PREC_NATIVE && (d->d_k == 128 || d->d_k == 64) && d->T >= kMinTensorT;
}
// head dimension the fp32 kernels work with on chip: 16 and 32 are zero-extended to 64
int simt_dim(const gka_desc *d) { return d->d_k <= 64 ? 64 : 128; }
long long work_units(const gka_desc *d) {
    return (long long)d->B * d->heads * (wants_tensor_path(d) ? tiles_of(d->T) : chunks_of(d->T));
}
// Upper bound on work items used for sizing (independent of the device).
int work_items_cap(const gka_desc *d, int chunk) {
    const long long nc = work_units(d);
    return (int)(nc < kMaxWorkItems ? nc : kMaxWorkItems);
}

}  // namespace
}  // namespace gka

using namespace gka;

extern "C" {

const char *gka_status_string(int status) {
    switch (status) {
        case GKA_OK: return "GKA_OK";
        case GKA_ERR_NULL: return "GKA_ERR_NULL: a required pointer is NULL";
        case GKA_ERR_SHAPE: return "GKA_ERR_SHAPE: bad size (non-positive, or d_k != d_v)";
        case GKA_ERR_DTYPE: return "GKA_ERR_DTYPE: unknown io_dtype or precision";
        case GKA_ERR_UNSUPPORTED: return "GKA_ERR_UNSUPPORTED: shape or mode outside the supported set";
        case GKA_ERR_WORKSPACE: return "GKA_ERR_WORKSPACE: workspace missing, misaligned or too small";
        case GKA_ERR_DOMAIN: return "GKA_ERR_DOMAIN: input outside its domain";
        case GKA_ERR_CUDA: return "GKA_ERR_CUDA: a CUDA call failed";
        case GKA_ERR_TIMEOUT: return "GKA_ERR_TIMEOUT: a bounded device-side wait ran out";
        case GKA_ERR_ALIGN: return "GKA_ERR_ALIGN: a data pointer is not aligned as required (16 bytes for vectors and states, 4 for per-token scalars)";
        default: return "GKA_ERR_?: unknown status";
    }
}

size_t gka_fwd_workspace_bytes(const gka_desc *desc, int chunk) {
    if (check_fwd_shape(desc, chunk) != GKA_OK) return 0;
    if (wants_tensor_path(desc)) return tc_workspace_bytes_for(work_items_cap(desc, chunk), work_units(desc));
    return workspace_bytes_for(work_items_cap(desc, chunk), simt_dim(desc), simt_dim(desc));
}

int gka_fwd_num_work_items(const gka_desc *desc, int chunk) {
    gka_status s = check_fwd_shape(desc, chunk);
    if (s != GKA_OK) return -(int)s;
    const int sms = sm_count();
    if (sms <= 0) return -(int)GKA_ERR_CUDA;
    const int cap = work_items_cap(desc, chunk);
    if (wants_tensor_path(desc)) {
        // Where the ranges cut sequences the summary kernel reads all keys and values once more.  Ranges of whole
        // sequences (pairs / k work items of k sequences each, k the smallest divisor of the number of (sequence, head)
        // pairs that leaves at most one item per SM) need no summaries, but may leave SMs idle in the state kernel and
        // make its run of tiles longer.  Measured per 128-token tile and block: 2.94 us in the state kernel with whole
        // sequences (2.15 us where two blocks share an item, one per master: at most half as many items as SMs),
        // 5.12 us x pairs / SMs for the summary and state kernels with one range per SM, which also cost 28 us more
        // per call.
        const long long pairs = (long long)desc->B * desc->heads, n = tiles_of(desc->T);
        for (long long k = (pairs + sms - 1) / sms; k <= pairs && k <= 64; ++k) {
            if (pairs % k != 0 || pairs / k > cap) continue;
            const long long items = pairs / k;
            const double per_tile = 2 * items <= sms ? 2.15 : 2.94;
            if ((double)n * ((double)k * per_tile - 5.12 * (double)pairs / sms) < 28.0) return (int)items;
            break;
        }
    }
    return sms < cap ? sms : cap;
}

gka_status gka_fwd_work_range(const gka_desc *desc, int chunk, int num_items, int item,
                              long long *first_chunk, long long *end_chunk, int *cut_in,
                              int *cut_out) {
    gka_status s = check_fwd_shape(desc, chunk);
    if (s != GKA_OK) return s;
    if (!first_chunk || !end_chunk || !cut_in || !cut_out) return GKA_ERR_NULL;
    WorkPlan p;
    const bool tiles = wants_tensor_path(desc);       // that path plans in 128-token tiles = pairs of chunks
    if (tiles) p.set(desc->B * desc->heads, tiles_of(desc->T), num_items > 0 ? num_items : 1, false);
    else p.set(desc->B * desc->heads, chunks_of(desc->T), num_items > 0 ? num_items : 1);
    if (num_items <= 0 || num_items > p.NC || item < 0 || item >= num_items) return GKA_ERR_SHAPE;
    // a tile is two chunks (the last tile of a sequence with an odd number of chunks holds one)
    const long long N = chunks_of(desc->T);
    auto chunk_of = [&](long long f) { return tiles ? (f / p.N) * N + 2 * (f % p.N) : f; };
    *first_chunk = chunk_of(p.lo(item));
    *end_chunk = chunk_of(p.lo(item + 1));
    *cut_in = p.cut_in(item) ? 1 : 0;
    *cut_out = p.cut_out(item) ? 1 : 0;
    return GKA_OK;
}

static gka_status fwd_impl(const gka_desc *desc, const void *q, const void *k, const void *v,
                           const float *gate, const float *lam, int n_iter, int chunk, void *out,
                           float *state_out, bool solve_only) {
    gka_status s = check_fwd_shape(desc, chunk);
    if (s != GKA_OK) return s;
    if (!q || !k || !v || !gate || !lam || !out) return GKA_ERR_NULL;
    if (n_iter < 0) return GKA_ERR_SHAPE;
    // vectors and states move in 16-byte pieces; the per-token scalars are read and written one float at a time
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(state_out) ||
        !aligned16(desc->state_in) || !aligned4(gate) || !aligned4(lam) || !aligned4(desc->fro_out) ||
        !aligned4(desc->beta) || !aligned4(desc->alpha))
        return GKA_ERR_ALIGN;
    const size_t need = gka_fwd_workspace_bytes(desc, chunk);
    if (!desc->workspace || desc->workspace_bytes < need ||
        (reinterpret_cast<uintptr_t>(desc->workspace) & 255u) != 0)
        return GKA_ERR_WORKSPACE;
    const int G = gka_fwd_num_work_items(desc, chunk);
    if (G <= 0) return GKA_ERR_CUDA;

    FwdArgs a;
    a.q = q; a.k = k; a.v = v; a.gate = gate; a.lam = lam; a.out = out;
    a.state_out = state_out;
    a.state_in = desc->state_in;
    a.fro_out = desc->fro_out;
    a.beta = desc->beta;
    a.alpha = solve_only ? nullptr : desc->alpha;
    a.device_status = desc->device_status;
    a.B = desc->B; a.T = desc->T; a.heads = desc->heads;
    a.d = desc->d_k;
    a.divH.set((unsigned)desc->heads);
    a.n_iter = n_iter;
    a.flags = desc->flags;
    a.solve_only = solve_only ? 1 : 0;
    a.start_from_scan = 0;
    a.state_split = 0;
    a.after_summary = 0;
    const bool tensor_path = wants_tensor_path(desc) && fwd_tc_available();
    a.tile_hh = nullptr;
    a.tile_hu = nullptr;
    if (tensor_path) {
        a.plan.set(desc->B * desc->heads, tiles_of(desc->T), G, false);
        const TcWorkspace w = carve_tc_workspace(desc->workspace, G, a.plan.NC);
        a.ws.start = w.start;
        a.ws.delta = w.delta;
        a.ws.cur = nullptr;
        a.ws.decay = w.decay;
        a.tile_hh = w.hh;
        a.tile_hu = w.hu;
    } else {
        if (wants_tensor_path(desc)) return GKA_ERR_CUDA;   // no driver entry point for tensor maps
        a.plan.set(desc->B * desc->heads, chunks_of(desc->T), G);
        a.ws = carve_workspace(desc->workspace, G, simt_dim(desc), simt_dim(desc));
    }
    a.ev_start = reinterpret_cast<cudaEvent_t>(desc->profile_start);
    a.ev_stop = reinterpret_cast<cudaEvent_t>(desc->profile_stop);
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(desc->stream);

    cudaError_t err = launch_validate(desc, gate, lam, (size_t)desc->B * desc->T * desc->heads, stream);
    if (err != cudaSuccess) return cuda_result(err, "gka_fwd_chunked (validation pass)");
    if (tensor_path)
        err = launch_fwd_tc(a, stream);
    else
        err = launch_fwd_simt(a, desc->d_k, desc->io_dtype, stream);
    return cuda_result(err, tensor_path ? "gka_fwd_chunked (tensor-core path)" : "gka_fwd_chunked (fp32 path)");
}

gka_status gka_fwd_chunked(const gka_desc *desc, const void *q, const void *k, const void *v,
                           const float *gate, const float *lam, int n_iter, int chunk, void *out,
                           float *state_out) {
    return fwd_impl(desc, q, k, v, gate, lam, n_iter, chunk, out, state_out, false);
}

gka_status gka_solve_chunked(const gka_desc *desc, const void *rhs, const void *k, const float *gate,
                             const float *lam, int n_iter, int chunk, void *x_out) {
    if (desc && desc->d_k != desc->d_v) return GKA_ERR_SHAPE;
    // the value stream plays no part in the solve: the key tensor stands in for it
    return fwd_impl(desc, rhs, k, k, gate, lam, n_iter, chunk, x_out, nullptr, true);
}

gka_status gka_decode_step(const gka_desc *desc, float *state, const void *q, const void *k,
                           const void *v, const float *gate, const float *lam, int n_iter,
                           void *out) {
    gka_status s = check_desc_common(desc);
    if (s != GKA_OK) return s;
    if (!state || !q || !k || !v || !gate || !lam || !out) return GKA_ERR_NULL;
    if (n_iter < 0) return GKA_ERR_SHAPE;
    if (!aligned16(state) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
        return GKA_ERR_ALIGN;
    cudaError_t err = launch_validate(desc, gate, lam, (size_t)desc->B * desc->heads, reinterpret_cast<cudaStream_t>(desc->stream));
    if (err != cudaSuccess) return cuda_result(err, "gka_decode_step (validation pass)");
    if (desc->d_k < 64)      // small head dimensions: one warp per (sequence, head) pair
        err = launch_decode_small(state, q, k, v, gate, lam, n_iter, out, desc->B, 1, desc->heads, desc->d_k, desc->io_dtype,
                                  desc->flags, desc->beta, desc->alpha, reinterpret_cast<cudaEvent_t>(desc->profile_start),
                                  reinterpret_cast<cudaEvent_t>(desc->profile_stop), reinterpret_cast<cudaStream_t>(desc->stream));
    else
        err = launch_decode(state, q, k, v, gate, lam, n_iter, out, desc->B, desc->heads,
                                    desc->d_k, desc->io_dtype, desc->flags, desc->beta, desc->alpha, desc->device_status,
                                    reinterpret_cast<cudaEvent_t>(desc->profile_start),
                                    reinterpret_cast<cudaEvent_t>(desc->profile_stop),
                                    reinterpret_cast<cudaStream_t>(desc->stream));
    return cuda_result(err, "gka_decode_step");
}

gka_status gka_decode_tokens(const gka_desc *desc, float *state, const void *q, const void *k,
                             const void *v, const float *gate, const float *lam, int n_iter,
                             void *out) {
    gka_status s = check_desc_common(desc);
    if (s != GKA_OK) return s;
    if (!state || !q || !k || !v || !gate || !lam || !out) return GKA_ERR_NULL;
    if (n_iter < 0 || desc->T < 1) return GKA_ERR_SHAPE;
    if (!aligned16(state) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
        return GKA_ERR_ALIGN;
    if (desc->T == 1)      // one token: the single-step kernel (same layouts) overlaps the state write-back better
        return gka_decode_step(desc, state, q, k, v, gate, lam, n_iter, out);
    cudaError_t err = launch_validate(desc, gate, lam, (size_t)desc->B * desc->T * desc->heads, reinterpret_cast<cudaStream_t>(desc->stream));
    if (err != cudaSuccess) return cuda_result(err, "gka_decode_tokens (validation pass)");
    if (desc->d_k < 64)
        err = launch_decode_small(state, q, k, v, gate, lam, n_iter, out, desc->B, desc->T, desc->heads, desc->d_k, desc->io_dtype,
                                  desc->flags, desc->beta, desc->alpha, reinterpret_cast<cudaEvent_t>(desc->profile_start),
                                  reinterpret_cast<cudaEvent_t>(desc->profile_stop), reinterpret_cast<cudaStream_t>(desc->stream));
    else
        err = launch_decode_multi(state, q, k, v, gate, lam, n_iter, out, desc->B, desc->T, desc->heads,
                                          desc->d_k, desc->io_dtype, desc->flags, desc->beta, desc->alpha,
                                          desc->device_status,
                                          reinterpret_cast<cudaEvent_t>(desc->profile_start),
                                          reinterpret_cast<cudaEvent_t>(desc->profile_stop),
                                          reinterpret_cast<cudaStream_t>(desc->stream));
    return cuda_result(err, "gka_decode_tokens");
}

const char *gka_last_error_detail(void) { return g_detail; }

gka_status gka_selftest_bounded_wait(const gka_desc *desc, int polls) {
    if (!desc || !desc->device_status) return GKA_ERR_NULL;
    if (polls < 1 || polls > (1 << 20)) return GKA_ERR_SHAPE;
    bounded_wait_selftest_kernel<<<1, 128, 0, reinterpret_cast<cudaStream_t>(desc->stream)>>>(polls, desc->device_status);
    return cuda_result(cudaGetLastError(), "gka_selftest_bounded_wait");
}

static size_t align256(size_t n) { return (n + 255) / 256 * 256; }

size_t gka_fwd_host_staging_bytes(const gka_desc *desc) {
    if (check_desc_common(desc) != GKA_OK || desc->T <= 0) return 0;
    const size_t es = desc->io_dtype == GKA_BF16 ? 2 : 4;
    const size_t tok = (size_t)desc->B * desc->T * desc->heads;
    const size_t st = (size_t)desc->B * desc->heads * state_floats(desc->d_k, desc->d_v) * sizeof(float);
    const size_t carry = 2 * (size_t)desc->heads * state_floats(desc->d_k, desc->d_v) * sizeof(float);
    return 2 * align256(tok * desc->d_k * es) + 2 * align256(tok * desc->d_v * es) + 2 * align256(tok * 4) +
           align256(st) + align256(carry);
}

namespace {
// Helper streams and events of the host-buffer entry point, one set per device, created on first use and
// kept for the life of the process.
struct HostPipe {
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, done = nullptr;
    std::vector<cudaEvent_t> copied, computed;
};
std::mutex g_pipe_mutex;
HostPipe g_pipes[64];

cudaError_t get_pipe(int slices, HostPipe **pipe) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    HostPipe &hp = g_pipes[dev];
    if (!hp.in) {
        if ((err = cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking)) != cudaSuccess) return err;
        if ((err = cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking)) != cudaSuccess) return err;
        if ((err = cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming)) != cudaSuccess) return err;
        if ((err = cudaEventCreateWithFlags(&hp.done, cudaEventDisableTiming)) != cudaSuccess) return err;
    }
    while ((int)hp.copied.size() < slices) {
        cudaEvent_t e0, e1;
        if ((err = cudaEventCreateWithFlags(&e0, cudaEventDisableTiming)) != cudaSuccess) return err;
        if ((err = cudaEventCreateWithFlags(&e1, cudaEventDisableTiming)) != cudaSuccess) return err;
        hp.copied.push_back(e0);
        hp.computed.push_back(e1);
    }
    *pipe = &hp;
    return cudaSuccess;
}
}  // namespace

gka_status gka_fwd_chunked_host(const gka_desc *desc, void *staging, const void *q, const void *k,
                                const void *v, const float *gate, const float *lam, int n_iter,
                                int chunk, void *out, float *state_out) {
    gka_status s = check_fwd_shape(desc, chunk);
    if (s != GKA_OK) return s;
    if (!staging || !q || !k || !v || !gate || !lam || !out) return GKA_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(staging) & 255u) != 0) return GKA_ERR_ALIGN;
    const size_t es = desc->io_dtype == GKA_BF16 ? 2 : 4;
    const size_t tok = (size_t)desc->B * desc->T * desc->heads;
    const size_t nqk = tok * desc->d_k * es, nv = tok * desc->d_v * es, ng = tok * 4;
    const size_t st_floats = state_floats(desc->d_k, desc->d_v);
    unsigned char *p = reinterpret_cast<unsigned char *>(staging);
    unsigned char *dq = p; p += align256(nqk);
    unsigned char *dk = p; p += align256(nqk);
    unsigned char *dv = p; p += align256(nv);
    unsigned char *dout = p; p += align256(nv);
    unsigned char *dgate = p; p += align256(ng);
    unsigned char *dlam = p; p += align256(ng);
    float *dstate = reinterpret_cast<float *>(p); p += align256((size_t)desc->B * desc->heads * st_floats * sizeof(float));
    float *dcarry = reinterpret_cast<float *>(p);            // two states of one batch entry, for the pieces of a sequence
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(desc->stream);

    // Sequences are independent, so the batch is cut into slices that move through three stages on three
    // streams: copies in (helper stream), kernels (the caller's stream), copies out (second helper stream).
    // The two copy directions and the kernels overlap; the caller's stream ends up waiting for everything.
    // What the pipeline cannot hide is its tail, the kernels and the copy out of the last piece, so the last
    // batch entries are also cut along the sequence (the state is carried from piece to piece on the device).
    struct Job { int b0, nb, t0, tn; bool first, last; };
    std::vector<Job> jobs;
    const int per = (desc->B + 7) / 8;                       // at most 8 batch slices
    const int nslices = (desc->B + per - 1) / per;
    // pieces of the sequences of the last slice: two halves measured best (every further piece costs about as much
    // as it takes off the tail)
    const int tpieces = (desc->T >= 4 * 2 * kChunk) ? 2 : 1;
    for (int i = 0; i < nslices; ++i) {
        const int b0 = i * per, nb = (b0 + per <= desc->B) ? per : desc->B - b0;
        if (i + 1 < nslices || tpieces == 1) {
            jobs.push_back({b0, nb, 0, desc->T, true, true});
        } else {
            const int tstep = ((desc->T / tpieces + 2 * kChunk - 1) / (2 * kChunk)) * (2 * kChunk);   // whole 128-token tiles
            for (int b = b0; b < b0 + nb; ++b) {
                for (int t0 = 0; t0 < desc->T; t0 += tstep)
                    jobs.push_back({b, 1, t0, (t0 + tstep < desc->T) ? tstep : desc->T - t0, t0 == 0, t0 + tstep >= desc->T});
            }
        }
    }
    const int njobs = (int)jobs.size();
    HostPipe *hp = nullptr;
    cudaError_t err = get_pipe(njobs, &hp);
    if (err != cudaSuccess) return cuda_result(err, "gka_fwd_chunked_host (helper streams)");
    if ((err = cudaEventRecord(hp->start, stream)) != cudaSuccess ||
        (err = cudaStreamWaitEvent(hp->in, hp->start, 0)) != cudaSuccess ||
        (err = cudaStreamWaitEvent(hp->out, hp->start, 0)) != cudaSuccess)
        return cuda_result(err, "gka_fwd_chunked_host (stream ordering)");
    const size_t hh = (size_t)desc->heads;
    auto copy = [&](unsigned char *dst, const void *src, size_t off, size_t bytes, cudaMemcpyKind kind, cudaStream_t on) {
        return kind == cudaMemcpyHostToDevice
                   ? cudaMemcpyAsync(dst + off, static_cast<const unsigned char *>(src) + off, bytes, kind, on)
                   : cudaMemcpyAsync(static_cast<unsigned char *>(const_cast<void *>(src)) + off, dst + off, bytes, kind, on);
    };
    for (int i = 0; i < njobs; ++i) {
        const Job &j = jobs[i];
        // a job's tokens are one contiguous range: whole batch entries, or a token range of one entry
        const size_t tok0 = ((size_t)j.b0 * desc->T + j.t0) * hh, ntok = (size_t)j.nb * j.tn * hh;
        err = copy(dq, q, tok0 * desc->d_k * es, ntok * desc->d_k * es, cudaMemcpyHostToDevice, hp->in);
        if (err == cudaSuccess) err = copy(dk, k, tok0 * desc->d_k * es, ntok * desc->d_k * es, cudaMemcpyHostToDevice, hp->in);
        if (err == cudaSuccess) err = copy(dv, v, tok0 * desc->d_v * es, ntok * desc->d_v * es, cudaMemcpyHostToDevice, hp->in);
        if (err == cudaSuccess) err = copy(dgate, gate, tok0 * 4, ntok * 4, cudaMemcpyHostToDevice, hp->in);
        if (err == cudaSuccess) err = copy(dlam, lam, tok0 * 4, ntok * 4, cudaMemcpyHostToDevice, hp->in);
        if (err == cudaSuccess) err = cudaEventRecord(hp->copied[i], hp->in);
        if (err != cudaSuccess) return cuda_result(err, "gka_fwd_chunked_host (host-to-device copies)");
    }
    int carry = 0;
    for (int i = 0; i < njobs; ++i) {
        const Job &j = jobs[i];
        const size_t tok0 = ((size_t)j.b0 * desc->T + j.t0) * hh, ntok = (size_t)j.nb * j.tn * hh;
        const size_t ost = (size_t)j.b0 * hh * st_floats;
        if ((err = cudaStreamWaitEvent(stream, hp->copied[i], 0)) != cudaSuccess)
            return cuda_result(err, "gka_fwd_chunked_host (stream ordering)");
        gka_desc sub = *desc;
        sub.B = j.nb;
        sub.T = j.tn;
        // the first piece of a sequence starts from the caller's state (or zero), the others from the state the
        // piece before left in the carry buffer; the last one writes the caller's state_out
        if (j.first) sub.state_in = desc->state_in ? desc->state_in + ost : nullptr;
        else sub.state_in = dcarry + (size_t)carry * hh * st_floats;
        float *piece_state = j.last ? (state_out ? dstate + ost : nullptr) : dcarry + (size_t)(carry ^ 1) * hh * st_floats;
        if (!j.last) carry ^= 1;
        if (desc->fro_out) sub.fro_out = desc->fro_out + tok0;
        if (desc->beta) sub.beta = desc->beta + tok0;
        if (desc->alpha) sub.alpha = desc->alpha + tok0;
        if (i > 0) sub.profile_start = sub.profile_stop = nullptr;
        s = gka_fwd_chunked(&sub, dq + tok0 * desc->d_k * es, dk + tok0 * desc->d_k * es, dv + tok0 * desc->d_v * es,
                            reinterpret_cast<const float *>(dgate + tok0 * 4), reinterpret_cast<const float *>(dlam + tok0 * 4),
                            n_iter, chunk, dout + tok0 * desc->d_v * es, piece_state);
        if (s != GKA_OK) return s;
        err = cudaEventRecord(hp->computed[i], stream);
        if (err == cudaSuccess) err = cudaStreamWaitEvent(hp->out, hp->computed[i], 0);
        if (err == cudaSuccess) err = copy(dout, out, tok0 * desc->d_v * es, ntok * desc->d_v * es, cudaMemcpyDeviceToHost, hp->out);
        if (err == cudaSuccess && state_out && j.last)
            err = cudaMemcpyAsync(state_out + ost, dstate + ost, (size_t)j.nb * hh * st_floats * sizeof(float),
                                  cudaMemcpyDeviceToHost, hp->out);
        if (err != cudaSuccess) return cuda_result(err, "gka_fwd_chunked_host (device-to-host copies)");
    }
    err = cudaEventRecord(hp->done, hp->out);
    if (err == cudaSuccess) err = cudaStreamWaitEvent(stream, hp->done, 0);
    return cuda_result(err, "gka_fwd_chunked_host (stream ordering)");
}

}  // extern "C"
