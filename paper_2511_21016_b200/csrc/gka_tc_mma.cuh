// Operand tiles and tcgen05.mma issue helpers shared by the tensor-core kernels of the chunked GKA forward.
//
// Every operand is a [128 rows][128 columns] bf16 tile stored as two TMA boxes of [128 rows][64 columns] with the
// 128-byte swizzle, 16384 bytes apart.  The same bytes serve as a K-major operand (contraction over the columns)
// or as an MN-major operand (contraction over the rows) without a transposed copy.
#pragma once
#include "gka_tc_util.cuh"

namespace gka {
namespace tcu {

constexpr uint32_t kTileBytes = 32768;

// byte offset of the 16-byte group holding columns 8 g .. 8 g + 7 (g = 0..15) of row r
__device__ __forceinline__ uint32_t tile_off(int r, int g) {
    return (uint32_t)((g >> 3) * 16384 + r * 128 + (((g & 7) ^ (r & 7)) << 4));
}

// ---- descriptor low words relative to (shared base >> 4); k-steps of 16
__host__ __device__ constexpr uint32_t t_kmaj(uint32_t off) { return (off >> 4) | ((16u >> 4) << 16); }
__host__ __device__ constexpr uint32_t t_mn(uint32_t off) { return (off >> 4) | ((16384u >> 4) << 16); }
__host__ __device__ constexpr uint32_t t_kstep(int ks) { return (uint32_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4); }
__host__ __device__ constexpr uint32_t t_mnstep(int ks) { return (uint32_t)((ks * 2048) >> 4); }

// D (+)= A x B, both operands in shared memory: low words are a base register plus an immediate
template <int ACC, uint32_t A_CONST, uint32_t B_CONST>
__device__ __forceinline__ void mma_ss2(uint32_t d_tmem, uint32_t a_base, uint32_t b_base, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .b64 da, db;\n\t.reg .b32 la, lb;\n\t"
        "add.u32 la, %1, %5;\n\tadd.u32 lb, %2, %6;\n\t"
        "mov.b64 da, {la, %4};\n\tmov.b64 db, {lb, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, %7;\n\t}" ::"r"(d_tmem), "r"(a_base), "r"(b_base), "r"(idesc),
        "r"(kDescHi), "n"(A_CONST), "n"(B_CONST), "n"(ACC)
        : "memory");
}
// D += A x B with A (packed bf16 pairs) in TMEM
template <uint32_t B_CONST>
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_base, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .b64 db;\n\t.reg .b32 lb;\n\t.reg .pred p;\n\t"
        "add.u32 lb, %2, %5;\n\tmov.b64 db, {lb, %4};\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, p;\n\t}" ::"r"(d_tmem), "r"(a_tmem), "r"(b_base), "r"(idesc),
        "r"(kDescHi), "n"(B_CONST)
        : "memory");
}
template <int ACC0, int NK = 8, int KS = 0>   // both K-major, NK k-steps over the first 16 NK columns
__device__ __forceinline__ void mma8_kk(uint32_t d, uint32_t a_base, uint32_t b_base, uint32_t idesc) {
    if constexpr (KS < NK) {
        mma_ss2<(KS == 0 ? ACC0 : 1), t_kmaj(0) + t_kstep(KS), t_kmaj(0) + t_kstep(KS)>(d, a_base, b_base, idesc);
        mma8_kk<ACC0, NK, KS + 1>(d, a_base, b_base, idesc);
    }
}
template <int ACC0, int KS = 0>   // both MN-major, 8 k-steps over the 128 rows
__device__ __forceinline__ void mma8_mm(uint32_t d, uint32_t a_base, uint32_t b_base, uint32_t idesc) {
    if constexpr (KS < 8) {
        mma_ss2<(KS == 0 ? ACC0 : 1), t_mn(0) + t_mnstep(KS), t_mn(0) + t_mnstep(KS)>(d, a_base, b_base, idesc);
        mma8_mm<ACC0, KS + 1>(d, a_base, b_base, idesc);
    }
}
// A = packed bf16 in TMEM: key block cq (32 keys) sits in the first 16 columns of the 32-column block cq of the
// score accumulator, so k-step ks (16 keys) reads columns 32 (ks / 2) + 8 (ks % 2).  B MN-major.  Accumulates.
template <int KS = 0>
__device__ __forceinline__ void mma8_pm(uint32_t d, uint32_t p_tmem, uint32_t b_base, uint32_t idesc) {
    if constexpr (KS < 8) {
        mma_ts<t_mn(0) + t_mnstep(KS)>(d, p_tmem + 32 * (KS >> 1) + 8 * (KS & 1), b_base, idesc);
        mma8_pm<KS + 1>(d, p_tmem, b_base, idesc);
    }
}
// D += A x B with A in TMEM, the lane quadrants below QLO of D left untouched (their rows of A need not be valid)
template <uint32_t B_CONST, int QLO>
__device__ __forceinline__ void mma_ts_rows(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_base, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .b64 db;\n\t.reg .b32 lb;\n\t.reg .pred p;\n\t"
        "add.u32 lb, %2, %5;\n\tmov.b64 db, {lb, %4};\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, {%6, %7, %8, %9}, p;\n\t}" ::"r"(d_tmem), "r"(a_tmem), "r"(b_base),
        "r"(idesc), "r"(kDescHi), "n"(B_CONST), "r"(QLO > 0 ? 0xFFFFFFFFu : 0u), "r"(QLO > 1 ? 0xFFFFFFFFu : 0u),
        "r"(QLO > 2 ? 0xFFFFFFFFu : 0u), "r"(0u)
        : "memory");
}
// P Khat with the masked scores of key block kb valid only for the lane quadrants kb .. 3 (tokens below see none of its keys)
template <int KS = 0>
__device__ __forceinline__ void mma8_pm_rows(uint32_t d, uint32_t p_tmem, uint32_t b_base, uint32_t idesc) {
    if constexpr (KS < 8) {
        mma_ts_rows<t_mn(0) + t_mnstep(KS), (KS >> 1)>(d, p_tmem + 32 * (KS >> 1) + 8 * (KS & 1), b_base, idesc);
        mma8_pm_rows<KS + 1>(d, p_tmem, b_base, idesc);
    }
}

constexpr uint32_t kIdescKK = make_idesc(128, 128, 0, 0);   // both operands K-major
constexpr uint32_t kIdescPM = make_idesc(128, 128, 0, 1);   // A from TMEM, B MN-major
constexpr uint32_t kIdescMM = make_idesc(128, 128, 1, 1);   // both MN-major

#define TMEM_ST8(taddr, r)                                                                                       \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(r[0]), \
                 "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])                     \
                 : "memory")

// TMA: one [128 rows][128 columns] operand tile = two boxes of 64 columns, the second one at column x_hi; `bar` gets
// 32768 bytes of transactions.  With head dimension 64 the second box lies past the last column of the tensor and
// reads as zeros (the tile is the head's rows zero-extended to 128 channels).
__device__ __forceinline__ void tma_load_tile3(const CUtensorMap *map, uint32_t dst, uint32_t bar, int x, int x_hi, int y, int z) {
#pragma unroll
    for (int hf = 0; hf < 2; ++hf)
        asm volatile(
            "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::
                "r"(dst + 16384 * hf), "l"(reinterpret_cast<uint64_t>(map)), "r"(hf ? x_hi : x), "r"(y), "r"(z), "r"(bar)
            : "memory");
}
// column of the second box of head h's tile: the head's upper 64 channels, or past the tensor for head dimension 64
__host__ __device__ __forceinline__ int tile_x_hi(int h, int d, int heads) { return d == 128 ? h * 128 + 64 : heads * d; }
__device__ __forceinline__ void tma_load_tile2(const CUtensorMap *map, uint32_t dst, uint32_t bar, int y) {
#pragma unroll
    for (int hf = 0; hf < 2; ++hf)
        asm volatile(
            "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::
                "r"(dst + 16384 * hf), "l"(reinterpret_cast<uint64_t>(map)), "r"(64 * hf), "r"(y), "r"(bar)
            : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

// 2-D map over the per-tile bf16 state copies: rows of 128 columns, box = 64 columns x 128 rows, 128-byte swizzle
inline bool make_state_map(CUtensorMap *map, const void *base, unsigned long long rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {128, (cuuint64_t)rows};
    cuuint64_t strides[1] = {256};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tcu
}  // namespace gka
