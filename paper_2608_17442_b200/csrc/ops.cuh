// Internal interfaces between the ciphertext-operation translation units.
#pragma once
#include "common.cuh"

// Scratch of one key-switch chunk (all [chunk][...][N] words):
//   dcoef [level]            the polynomial being switched, transformed to COEFF in place
//   ext   [beta][level+K]    converted digits; the rows of a digit's own limbs hold the polynomial itself (EVAL);
//                            n_ext such buffers in a row when several polynomials are switched before one sum
//   acc   [2][level+K]       inner-product accumulators
//   u     [2][level]         converted special-limb part
struct KsScratch {
    u64 *dcoef, *ext, *acc, *u;
};
size_t ks_scratch_words(const fesc_ctx* ctx, uint32_t level, uint32_t chunk, uint32_t n_ext = 1);
KsScratch ks_scratch_carve(const fesc_ctx* ctx, u64* base, uint32_t level, uint32_t chunk, uint32_t n_ext = 1);
// converted polynomials a deferred giant-step sum of n_terms keeps side by side (one inner-product pass over them)
static inline uint32_t giant_ext_buffers(uint32_t n_terms) { return n_terms < 2 ? 1 : (n_terms - 1 < 4 ? n_terms - 1 : 4); }
uint32_t ks_chunk(const fesc_ctx* ctx, uint32_t batch);

int rotate_internal(fesc_ctx* ctx, const u64* in, size_t in_stride, u64* out, size_t out_stride, uint32_t batch,
                    uint32_t level, uint32_t key_id, u64* scratch, cudaStream_t st, int accumulate);
int rotate_hoisted_internal(fesc_ctx* ctx, const u64* in, size_t in_stride, u64* out, size_t out_stride,
                            size_t key_stride, uint32_t batch, uint32_t level, const uint32_t* key_ids, uint32_t n_keys,
                            u64* scratch, cudaStream_t st);
int rotate_sum_hoisted_internal(fesc_ctx* ctx, const u64* in, size_t in_stride, u64* out, size_t out_stride,
                                uint32_t batch, uint32_t level, const uint32_t* key_ids, uint32_t n_keys, u64* scratch,
                                cudaStream_t st);
// scratch: ks_scratch_words(ctx, level, ks_chunk(ctx, batch), giant_ext_buffers(n_terms)) words
int giant_sum_deferred_internal(fesc_ctx* ctx, u64* acc, uint32_t n_terms, size_t ct_words, uint32_t batch,
                                uint32_t level, uint32_t key_base, u64* scratch, cudaStream_t st);
int rescale_internal(fesc_ctx* ctx, const u64* in, size_t in_stride, u64* out, uint32_t batch, uint32_t level,
                     u64* scratch, cudaStream_t st);
int ctmul_internal(fesc_ctx* ctx, const u64* a, size_t a_stride, const u64* b, size_t b_stride, u64* out,
                   size_t out_stride, uint32_t batch, uint32_t level, u64* scratch, cudaStream_t st);

// ---------------------------------------------------------------------------------------
// Byte-plane products on the tensor cores (BSGS accumulate): u8 x u8 -> s32 mma.sync m16n8k32 and the recombination
// of the 7 x 7 byte-plane sums of one output.
// ---------------------------------------------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ void imma_u8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// the same product with zero addends (first k-step of a tile).  z0..z3 are four registers that hold zero and are kept
// opaque to the optimiser, so that they stay one fixed operand quad instead of being rebuilt before every instruction.
__device__ __forceinline__ void imma_u8_zero(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1, int z0, int z1, int z2, int z3) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
                 : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(z0), "r"(z1), "r"(z2), "r"(z3));
}
// d[k] = (byte k of w0) | (byte k of w1) << 8 | (byte k of w2) << 16 | (byte k of w3) << 24, k = 0..6
__device__ __forceinline__ void byte_planes4(u64 w0, u64 w1, u64 w2, u64 w3, uint32_t (&d)[7]) {
    const uint32_t l0 = (uint32_t)w0, l1 = (uint32_t)w1, l2 = (uint32_t)w2, l3 = (uint32_t)w3;
    const uint32_t h0 = (uint32_t)(w0 >> 32), h1 = (uint32_t)(w1 >> 32), h2 = (uint32_t)(w2 >> 32), h3 = (uint32_t)(w3 >> 32);
    const uint32_t t0 = __byte_perm(l0, l1, 0x5140), t1 = __byte_perm(l2, l3, 0x5140);
    const uint32_t t2 = __byte_perm(l0, l1, 0x7362), t3 = __byte_perm(l2, l3, 0x7362);
    d[0] = __byte_perm(t0, t1, 0x5410);
    d[1] = __byte_perm(t0, t1, 0x7632);
    d[2] = __byte_perm(t2, t3, 0x5410);
    d[3] = __byte_perm(t2, t3, 0x7632);
    const uint32_t u0 = __byte_perm(h0, h1, 0x5140), u1 = __byte_perm(h2, h3, 0x5140);
    const uint32_t u2 = __byte_perm(h0, h1, 0x7362), u3 = __byte_perm(h2, h3, 0x7362);
    d[4] = __byte_perm(u0, u1, 0x5410);
    d[5] = __byte_perm(u0, u1, 0x7632);
    d[6] = __byte_perm(u2, u3, 0x5410);
}
// Recombination.  d[m][j][r]: accumulators of m-tile m (byte planes 2m, 2m+1 of the diagonal side), n-tile j (byte plane
// j of the input side); registers r = 0,1 belong to plane 2m and r = 2,3 to plane 2m+1, r & 1 = sel picks the polynomial.
// E_d = sum_{k+j=d} D[k][j] (13 values; below 2^28 for at most 512 terms), four of them are packed exactly into one
// integer T_m < 2^52, and S = T_0 + T_1 2^32 + T_2 2^64 + T_3 2^96 is reduced modulo q: with exact FP64 products for
// primes below 2^50 (|fp_reduce| <= q/2 and every lazy product within 2q, so the sum stays below 6.5 q < 2^53), as a
// 128-bit integer otherwise.  c32, c64, c96 = 2^32, 2^64, 2^96 mod q (FP path only).
template <bool FP>
__device__ __forceinline__ u64 imma_recombine(const int (&d)[4][7][4], int sel, const PrimeConst& pc, double c32, double c64,
                                              double c96) {
    uint32_t e[13];
#pragma unroll
    for (int x = 0; x < 13; x++) e[x] = 0;
#pragma unroll
    for (int k = 0; k < 7; k++)
#pragma unroll
        for (int j = 0; j < 7; j++) e[k + j] += (uint32_t)d[k >> 1][j][(k & 1) * 2 + sel];
    const u64 w0 = e[0] + ((u64)e[1] << 8) + ((u64)e[2] << 16) + ((u64)e[3] << 24);
    const u64 w1 = e[4] + ((u64)e[5] << 8) + ((u64)e[6] << 16) + ((u64)e[7] << 24);
    const u64 w2 = e[8] + ((u64)e[9] << 8) + ((u64)e[10] << 16) + ((u64)e[11] << 24);
    if (FP) {
        const double q = pc.qd, qinv = pc.qinvd;
        const double r = fp_reduce(fp_from_u64(w0), q, qinv) + fp_modmul(fp_from_u64(w1), c32, q, qinv) +
                         fp_modmul(fp_from_u64(w2), c64, q, qinv) + fp_modmul(fp_from_u64((u64)e[12]), c96, q, qinv);
        return fp_store(r, q, qinv);
    }
    const u128 S = (u128)w0 + ((u128)w1 << 32) + ((u128)w2 << 64) + ((u128)e[12] << 96);
    return reduce128((u64)(S >> 64), (u64)S, pc);
}
#endif

// basis conversions on the tensor cores (bconv.cu)
bool bconv_supported(const fesc_ctx* ctx, uint32_t level);
void moddown_conv_imma_launch(fesc_ctx* ctx, const u64* acc, u64* u, uint32_t level, uint32_t batch, int out_double, cudaStream_t st);

// packed-operand BSGS accumulate (packed.cu)
size_t bsgs_packed_bytes(uint32_t N, uint32_t level, uint32_t rows, uint32_t terms);
bool bsgs_packed_supported(const fesc_ctx* ctx, uint32_t level, uint32_t terms, uint32_t dshift);
int bsgs_pack_inputs(fesc_ctx* ctx, const u64* rot, uint8_t* xpk, uint32_t level, uint32_t tbs, uint32_t terms, cudaStream_t st);
int bsgs_accumulate_packed(fesc_ctx* ctx, const uint8_t* xpk, const uint8_t* dpk, u64* acc, uint32_t level, uint32_t tbs,
                           uint32_t terms, uint32_t bp_count, bool fp, uint32_t dshift, cudaStream_t st);
