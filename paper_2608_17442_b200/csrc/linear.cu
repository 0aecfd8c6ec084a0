// BSGS plaintext-weight projection Y = XW on packed ciphertexts.
//
// Per group of token blocks: (1) baby rotations of every input ciphertext, batched per rotation
// amount so a key is streamed once per batch; (2) one fused accumulate kernel that forms every
// giant-step accumulator acc[tb][b][p] = sum_{g,q} rot[tb][g][q] (.) D[b][p][g][q] exactly in
// registers (mixed integer/FP64 sums for primes below 2^50, exact FP64 products, or 128-bit lazy
// integer sums), tiled TT token blocks x PT (b,p) pairs per thread so a rotated
// ciphertext word is reused PT times and a diagonal word TT times; (3) giant rotations that
// accumulate straight into acc[tb][b][0] (optionally with one division by P for the whole sum);
// (4) rescale into the output.
#include <stdlib.h>
#include <string.h>

#include "ops.cuh"

template <int TT, int PT>
__global__ void __launch_bounds__(256, (TT * PT >= 16 ? 1 : (TT * PT >= 4 ? 2 : 3))) k_bsgs_accumulate(
    const u64* __restrict__ rot,    // [tbs][terms][2][level][N]   rotated inputs, term = g*n1 + q
    const u64* __restrict__ diags,  // [bp_count][terms][level][N]
    u64* __restrict__ acc,          // [tbs][bp_count][2][level][N]
    const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level, uint32_t tbs, uint32_t terms,
    uint32_t bp_count, uint32_t reduce_every) {
    // blockIdx.x walks the (b,p) tiles of one (coefficient tile, limb, token-block tile), so CTAs
    // that run together read the same ciphertext words: those come from HBM once and from L2 after.
    const uint32_t c = blockIdx.y * blockDim.x + threadIdx.x;
    const uint32_t l = blockIdx.z % level;
    const uint32_t tb0 = (blockIdx.z / level) * TT, bp0 = blockIdx.x * PT;
    if (c >= N) return;
    const PrimeConst pc = pcs[l];
    const size_t poly = (size_t)level * N, ctw = 2 * poly;
    const size_t o = (size_t)l * N + c;
    // out-of-range tile members recompute the last valid one and are not stored
    const u64* xp[TT];
    const u64* dp[PT];
#pragma unroll
    for (int i = 0; i < TT; i++) {
        uint32_t tb = tb0 + i < tbs ? tb0 + i : tbs - 1;
        xp[i] = rot + (size_t)tb * terms * ctw + o;
    }
#pragma unroll
    for (int j = 0; j < PT; j++) {
        uint32_t bp = bp0 + j < bp_count ? bp0 + j : bp_count - 1;
        dp[j] = diags + (size_t)bp * terms * poly + o;
    }
    acc128 a[TT][PT][2];
#pragma unroll
    for (int i = 0; i < TT; i++)
#pragma unroll
        for (int j = 0; j < PT; j++) a[i][j][0] = a[i][j][1] = acc128{0, 0};
    // software pipeline: operands of term t+1 are in flight while term t is multiplied
    u64 x0[TT], x1[TT], w[PT], nx0[TT], nx1[TT], nw[PT];
#pragma unroll
    for (int i = 0; i < TT; i++) {
        x0[i] = xp[i][0];
        x1[i] = xp[i][poly];
    }
#pragma unroll
    for (int j = 0; j < PT; j++) w[j] = __ldg(dp[j]);
    uint32_t since = 0;
#pragma unroll 1
    for (uint32_t t = 0; t < terms; t++) {
        const bool more = t + 1 < terms;
        const size_t xo = more ? (size_t)(t + 1) * ctw : (size_t)t * ctw;
        const size_t wo = more ? (size_t)(t + 1) * poly : (size_t)t * poly;
#pragma unroll
        for (int i = 0; i < TT; i++) {
            nx0[i] = xp[i][xo];
            nx1[i] = xp[i][xo + poly];
        }
#pragma unroll
        for (int j = 0; j < PT; j++) nw[j] = __ldg(dp[j] + wo);
#pragma unroll
        for (int j = 0; j < PT; j++)
#pragma unroll
            for (int i = 0; i < TT; i++) {
                mac128(a[i][j][0], x0[i], w[j]);
                mac128(a[i][j][1], x1[i], w[j]);
            }
        if (++since == reduce_every) {
            since = 0;
#pragma unroll
            for (int i = 0; i < TT; i++)
#pragma unroll
                for (int j = 0; j < PT; j++)
#pragma unroll
                    for (int p = 0; p < 2; p++) a[i][j][p] = acc128{reduce128(a[i][j][p].hi, a[i][j][p].lo, pc), 0};
        }
#pragma unroll
        for (int i = 0; i < TT; i++) {
            x0[i] = nx0[i];
            x1[i] = nx1[i];
        }
#pragma unroll
        for (int j = 0; j < PT; j++) w[j] = nw[j];
    }
#pragma unroll
    for (int i = 0; i < TT; i++)
#pragma unroll
        for (int j = 0; j < PT; j++) {
            const uint32_t tb = tb0 + i, bp = bp0 + j;
            if (tb < tbs && bp < bp_count) {
                u64* dst = acc + ((size_t)tb * bp_count + bp) * ctw;
                dst[o] = reduce128(a[i][j][0].hi, a[i][j][0].lo, pc);
                dst[poly + o] = reduce128(a[i][j][1].hi, a[i][j][1].lo, pc);
            }
        }
}

// The same accumulation on the FP64 pipe, for limbs whose primes are all below 2^50: every term is an
// exact signed lazy product (fp_modmul), partial sums stay below 2^53 because they are folded back to
// |acc| <= q/2 every 8 terms.  Accumulators are single doubles, so the 2 x 8 tile needs half the
// registers of the 128-bit version and two CTAs fit per SM.
template <int TT, int PT>
__global__ void __launch_bounds__(256, 2) k_bsgs_accumulate_fp(
    const u64* __restrict__ rot, const u64* __restrict__ diags, u64* __restrict__ acc,
    const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level, uint32_t tbs, uint32_t terms, uint32_t bp_count) {
    const uint32_t c = blockIdx.y * blockDim.x + threadIdx.x;
    const uint32_t l = blockIdx.z % level;
    const uint32_t tb0 = (blockIdx.z / level) * TT, bp0 = blockIdx.x * PT;
    if (c >= N) return;
    const double q = pcs[l].qd, qinv = pcs[l].qinvd;
    const size_t poly = (size_t)level * N, ctw = 2 * poly;
    const size_t o = (size_t)l * N + c;
    const u64* xp[TT];
    const u64* dp[PT];
#pragma unroll
    for (int i = 0; i < TT; i++) {
        uint32_t tb = tb0 + i < tbs ? tb0 + i : tbs - 1;
        xp[i] = rot + (size_t)tb * terms * ctw + o;
    }
#pragma unroll
    for (int j = 0; j < PT; j++) {
        uint32_t bp = bp0 + j < bp_count ? bp0 + j : bp_count - 1;
        dp[j] = diags + (size_t)bp * terms * poly + o;
    }
    double a[TT][PT][2];
#pragma unroll
    for (int i = 0; i < TT; i++)
#pragma unroll
        for (int j = 0; j < PT; j++) a[i][j][0] = a[i][j][1] = 0.0;
    u64 nx0[TT], nx1[TT], nw[PT];
#pragma unroll
    for (int i = 0; i < TT; i++) {
        nx0[i] = xp[i][0];
        nx1[i] = xp[i][poly];
    }
#pragma unroll
    for (int j = 0; j < PT; j++) nw[j] = __ldg(dp[j]);
#pragma unroll 1
    for (uint32_t t = 0; t < terms; t++) {
        double x0[TT], x1[TT], w[PT];
#pragma unroll
        for (int i = 0; i < TT; i++) {
            x0[i] = fp_load(nx0[i], q);
            x1[i] = fp_load(nx1[i], q);
        }
#pragma unroll
        for (int j = 0; j < PT; j++) w[j] = fp_from_u64(nw[j]);
        const uint32_t tn = t + 1 < terms ? t + 1 : t;
#pragma unroll
        for (int i = 0; i < TT; i++) {
            nx0[i] = xp[i][(size_t)tn * ctw];
            nx1[i] = xp[i][(size_t)tn * ctw + poly];
        }
#pragma unroll
        for (int j = 0; j < PT; j++) nw[j] = __ldg(dp[j] + (size_t)tn * poly);
#pragma unroll
        for (int j = 0; j < PT; j++)
#pragma unroll
            for (int i = 0; i < TT; i++) {
                a[i][j][0] += fp_modmul(x0[i], w[j], q, qinv);
                a[i][j][1] += fp_modmul(x1[i], w[j], q, qinv);
            }
        if ((t & 7) == 7) {
#pragma unroll
            for (int i = 0; i < TT; i++)
#pragma unroll
                for (int j = 0; j < PT; j++) {
                    a[i][j][0] = fp_reduce(a[i][j][0], q, qinv);
                    a[i][j][1] = fp_reduce(a[i][j][1], q, qinv);
                }
        }
    }
#pragma unroll
    for (int i = 0; i < TT; i++)
#pragma unroll
        for (int j = 0; j < PT; j++) {
            const uint32_t tb = tb0 + i, bp = bp0 + j;
            if (tb < tbs && bp < bp_count) {
                u64* dst = acc + ((size_t)tb * bp_count + bp) * ctw;
                dst[o] = fp_store(a[i][j][0], q, qinv);
                dst[poly + o] = fp_store(a[i][j][1], q, qinv);
            }
        }
}

// FP64 accumulate with asynchronous staging: every thread copies its own operand words of the next
// STAGES-1 terms into shared memory with cp.async (8 bytes each, no barrier: a thread only reads back what
// it copied), so several terms of operands are in flight per thread without holding them in registers.
__device__ __forceinline__ void cp_async8(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
                 : "memory");
}
__device__ __forceinline__ void cp_async8s(uint32_t smem_dst, const void* gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N_>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N_) : "memory");
}

template <int TT, int PT, int STAGES>
__global__ void __launch_bounds__(256, (TT * PT > 16 ? 1 : 2)) k_bsgs_accumulate_fp_staged(
    const u64* __restrict__ rot, const u64* __restrict__ diags, u64* __restrict__ acc,
    const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level, uint32_t tbs, uint32_t terms, uint32_t bp_count) {
    constexpr int ROWS = 2 * TT + PT;
    extern __shared__ __align__(16) u64 stage[];          // [STAGES][ROWS][256]
    const uint32_t tid = threadIdx.x;
    const uint32_t c = blockIdx.y * 256 + tid;            // N is a multiple of 256
    const uint32_t l = blockIdx.z % level;
    const uint32_t tb0 = (blockIdx.z / level) * TT, bp0 = blockIdx.x * PT;
    const double q = pcs[l].qd, qinv = pcs[l].qinvd;
    const size_t poly = (size_t)level * N, ctw = 2 * poly;
    const size_t o = (size_t)l * N + c;
    const u64* xp[TT];
    const u64* dp[PT];
#pragma unroll
    for (int i = 0; i < TT; i++) {
        uint32_t tb = tb0 + i < tbs ? tb0 + i : tbs - 1;
        xp[i] = rot + (size_t)tb * terms * ctw + o;
    }
#pragma unroll
    for (int j = 0; j < PT; j++) {
        uint32_t bp = bp0 + j < bp_count ? bp0 + j : bp_count - 1;
        dp[j] = diags + (size_t)bp * terms * poly + o;
    }
    auto issue = [&](uint32_t t) {
        u64* dst = stage + (size_t)(t % STAGES) * ROWS * 256 + tid;
#pragma unroll
        for (int i = 0; i < TT; i++) {
            cp_async8(dst + (2 * i) * 256, xp[i] + (size_t)t * ctw);
            cp_async8(dst + (2 * i + 1) * 256, xp[i] + (size_t)t * ctw + poly);
        }
#pragma unroll
        for (int j = 0; j < PT; j++) cp_async8(dst + (2 * TT + j) * 256, dp[j] + (size_t)t * poly);
    };
    for (uint32_t t = 0; t < STAGES - 1; t++) {
        if (t < terms) issue(t);
        cp_async_commit();
    }
    double a[TT][PT][2];
#pragma unroll
    for (int i = 0; i < TT; i++)
#pragma unroll
        for (int j = 0; j < PT; j++) a[i][j][0] = a[i][j][1] = 0.0;
#pragma unroll 1
    for (uint32_t t = 0; t < terms; t++) {
        if (t + STAGES - 1 < terms) issue(t + STAGES - 1);
        cp_async_commit();
        cp_async_wait<STAGES - 1>();                       // the group of term t has landed
        const u64* sm = stage + (size_t)(t % STAGES) * ROWS * 256 + tid;
        double x0[TT], x1[TT];
#pragma unroll
        for (int i = 0; i < TT; i++) {
            x0[i] = fp_load(sm[(2 * i) * 256], q);
            x1[i] = fp_load(sm[(2 * i + 1) * 256], q);
        }
#pragma unroll
        for (int j = 0; j < PT; j++) {
            const double w = fp_from_u64(sm[(2 * TT + j) * 256]);
#pragma unroll
            for (int i = 0; i < TT; i++) {
                a[i][j][0] += fp_modmul(x0[i], w, q, qinv);
                a[i][j][1] += fp_modmul(x1[i], w, q, qinv);
            }
        }
        if ((t & 7) == 7) {
#pragma unroll
            for (int i = 0; i < TT; i++)
#pragma unroll
                for (int j = 0; j < PT; j++) {
                    a[i][j][0] = fp_reduce(a[i][j][0], q, qinv);
                    a[i][j][1] = fp_reduce(a[i][j][1], q, qinv);
                }
        }
    }
#pragma unroll
    for (int i = 0; i < TT; i++)
#pragma unroll
        for (int j = 0; j < PT; j++) {
            const uint32_t tb = tb0 + i, bp = bp0 + j;
            if (tb < tbs && bp < bp_count) {
                u64* dst = acc + ((size_t)tb * bp_count + bp) * ctw;
                dst[o] = fp_store(a[i][j][0], q, qinv);
                dst[poly + o] = fp_store(a[i][j][1], q, qinv);
            }
        }
}

// Mixed-pipe exact accumulation for primes below 2^50 (at most 256 terms).  The sum S = sum_t x_t w_t
// (below 2^108) is tracked twice: its low 64 bits exactly on the integer multiplier pipe (one 32x32+64 and two
// 32-bit multiply-adds per term), and its magnitude approximately on the FP64 pipe (ONE fused multiply-add per
// term; every rounding is below 2^53, so 256 terms stay within 2^61 of S).  S is then the unique integer that is
// congruent to the low part modulo 2^64 and within 2^63 of the approximation; one 128-bit reduction follows.
// Per term that is 8 multiplier-pipe cycles and 2 FP64-pipe cycles per warp, on pipes that run concurrently,
// instead of 6 FP64 operations and a rounding.
// threads per CTA: two CTAs of 128 per SM (the registers allow 256 threads in all) overlap one CTA's reconstruction and
// stores with the other's term loop
#ifndef MIX_THREADS
#define MIX_THREADS 128
#endif
template <int TT, int PT, int STAGES>
__global__ void __launch_bounds__(MIX_THREADS, (TT * PT >= 12 ? 256 / MIX_THREADS : 2 * 256 / MIX_THREADS)) k_bsgs_accumulate_mixed(
    const u64* __restrict__ rot, const u64* __restrict__ diags, u64* __restrict__ acc,
    const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level, uint32_t tbs, uint32_t terms, uint32_t bp_count) {
    constexpr int ROWS = 2 * TT + PT;
    extern __shared__ __align__(16) u64 stage[];          // [STAGES][ROWS][MIX_THREADS]
    const uint32_t tid = threadIdx.x;
    const uint32_t c = blockIdx.y * MIX_THREADS + tid;
    // blockIdx.x = (b,p) tile * token-block tiles + token-block tile: CTAs that read the same diagonal rows are
    // scheduled next to each other (the second read hits L2), and so are the (b,p) tiles that share ciphertext rows
    const uint32_t tb_tiles = (tbs + TT - 1) / TT;
    const uint32_t l = blockIdx.z;
    const uint32_t tb0 = (blockIdx.x % tb_tiles) * TT, bp0 = (blockIdx.x / tb_tiles) * PT;
    const PrimeConst pc = pcs[l];
    const size_t poly = (size_t)level * N, ctw = 2 * poly;
    const size_t o = (size_t)l * N + c;
    // one running pointer per operand; the rows of a stage sit at block-uniform offsets from it
    size_t xoff[TT], doff[PT];
#pragma unroll
    for (int i = 0; i < TT; i++) xoff[i] = (size_t)(tb0 + i < tbs ? tb0 + i : tbs - 1) * terms * ctw;
#pragma unroll
    for (int j = 0; j < PT; j++) doff[j] = (size_t)(bp0 + j < bp_count ? bp0 + j : bp_count - 1) * terms * poly;
    const u64* xrun = rot + o;
    const u64* drun = diags + o;
    uint32_t slot = 0;                                     // stage that the next issue fills
    const uint32_t sbase = (uint32_t)__cvta_generic_to_shared(stage) + tid * 8;
    auto issue = [&]() {
        const uint32_t dst = sbase + slot * (ROWS * MIX_THREADS * 8);
#pragma unroll
        for (int i = 0; i < TT; i++) {
            cp_async8s(dst + (2 * i) * (MIX_THREADS * 8), xrun + xoff[i]);
            cp_async8s(dst + (2 * i + 1) * (MIX_THREADS * 8), xrun + xoff[i] + poly);
        }
#pragma unroll
        for (int j = 0; j < PT; j++) cp_async8s(dst + (2 * TT + j) * (MIX_THREADS * 8), drun + doff[j]);
        xrun += ctw;
        drun += poly;
        slot = slot + 1 == STAGES ? 0 : slot + 1;
    };
    for (uint32_t t = 0; t < STAGES - 1; t++) {
        if (t < terms) issue();
        cp_async_commit();
    }
    u64 lo[TT][PT][2];        // S mod 2^64 (low product word accumulated with wrap-around)
    uint32_t hi[TT][PT][2];   // cross terms, weight 2^32, modulo 2^32
    double ap[TT][PT][2];     // S approximately
#pragma unroll
    for (int i = 0; i < TT; i++)
#pragma unroll
        for (int j = 0; j < PT; j++)
#pragma unroll
            for (int p = 0; p < 2; p++) lo[i][j][p] = 0, hi[i][j][p] = 0, ap[i][j][p] = 0.0;
    uint32_t rslot = 0;                                    // stage that the next term reads
#pragma unroll 1
    for (uint32_t t = 0; t < terms; t++) {
        if (t + STAGES - 1 < terms) issue();
        cp_async_commit();
        cp_async_wait<STAGES - 1>();
        const u64* sm = stage + (size_t)rslot * ROWS * MIX_THREADS + tid;
        rslot = rslot + 1 == STAGES ? 0 : rslot + 1;
        uint32_t x0[TT][2], x1[TT][2];
        double xd[TT][2];
#pragma unroll
        for (int i = 0; i < TT; i++)
#pragma unroll
            for (int p = 0; p < 2; p++) {
                const u64 v = sm[(2 * i + p) * MIX_THREADS];
                x0[i][p] = (uint32_t)v;
                x1[i][p] = (uint32_t)(v >> 32);
                xd[i][p] = __ull2double_rn(v);       // exact: v < 2^50
            }
#pragma unroll
        for (int j = 0; j < PT; j++) {
            const u64 v = sm[(2 * TT + j) * MIX_THREADS];
            const uint32_t w0 = (uint32_t)v, w1 = (uint32_t)(v >> 32);
            const double wd = __ull2double_rn(v);
#pragma unroll
            for (int i = 0; i < TT; i++)
#pragma unroll
                for (int p = 0; p < 2; p++) {
                    asm("mad.wide.u32 %0, %1, %2, %0;" : "+l"(lo[i][j][p]) : "r"(x0[i][p]), "r"(w0));
                    asm("mad.lo.u32 %0, %1, %2, %0;" : "+r"(hi[i][j][p]) : "r"(x1[i][p]), "r"(w0));
                    asm("mad.lo.u32 %0, %1, %2, %0;" : "+r"(hi[i][j][p]) : "r"(x0[i][p]), "r"(w1));
                    ap[i][j][p] = __fma_rn(xd[i][p], wd, ap[i][j][p]);
                }
        }
    }
#pragma unroll
    for (int i = 0; i < TT; i++)
#pragma unroll
        for (int j = 0; j < PT; j++) {
            const uint32_t tb = tb0 + i, bp = bp0 + j;
            if (tb < tbs && bp < bp_count) {
                u64* dst = acc + ((size_t)tb * bp_count + bp) * ctw;
#pragma unroll
                for (int p = 0; p < 2; p++) {
                    const u64 low = lo[i][j][p] + ((u64)hi[i][j][p] << 32);
                    // the high word of S: round((approximation - low) / 2^64)
                    const double k = rint((ap[i][j][p] - __ull2double_rn(low)) * 5.421010862427522e-20);
                    dst[p * poly + o] = reduce128((u64)__double2ll_rn(k), low, pc);
                }
            }
        }
}

// Knobs for experiments.  FESC_BSGS_KERNEL picks the accumulate kernel: "int" the 128-bit integer one, "fp" the
// exact-FP64 one, anything else the default (mixed-pipe where it applies).  FESC_BSGS_GROUP_GIB fixes the scratch
// budget that decides how many token blocks are processed per group (default: from the free device memory).
static int bsgs_kernel() {
    static int v = -1;
    if (v < 0) {
        const char* e = getenv("FESC_BSGS_KERNEL");
        v = !e ? 0 : (!strcmp(e, "int") ? 2 : (!strcmp(e, "fp") ? 1 : 0));
    }
    return v;
}
// Larger groups re-read the diagonals less often and give the key-switch kernels larger batches; every token block
// of a group needs its rotated inputs and its partial sums resident.  Budget: 60% of what is free (counting the
// scratch arena the context already holds), between 2 and 24 GiB.
static size_t bsgs_group_bytes(fesc_ctx* ctx) {
    const char* e = getenv("FESC_BSGS_GROUP_GIB");
    if (e && atoi(e) > 0) return (size_t)atoi(e) << 30;
    size_t free_b = 0, total_b = 0;
    if (cudaMemGetInfo(&free_b, &total_b) != cudaSuccess) return (size_t)12 << 30;
    size_t budget = (free_b + ctx->scratch_bytes) / 10 * 6;
    const size_t lo = (size_t)2 << 30, hi = (size_t)24 << 30;
    return budget < lo ? lo : (budget > hi ? hi : budget);
}

extern "C" int fesc_linear(fesc_ctx* ctx, const uint64_t* d_ct_in, const uint64_t* d_diags, const fesc_bsgs_desc* desc,
                           uint64_t* d_ct_out, void* stream) {
    if (!ctx || !d_ct_in || !d_diags || !desc || !d_ct_out) return FESC_EINVAL;
    const uint32_t n1 = desc->n1, n2 = desc->n2, gin = desc->in_blocks, nout = desc->out_blocks;
    const uint32_t tbs = desc->token_blocks, level = desc->n_limbs, N = ctx->N;
    if (!n1 || !n2 || !gin || !nout || !tbs) return fesc_fail(ctx, FESC_EINVAL, "linear: empty dimension");
    if (level < 2 || level > ctx->n_q) return fesc_fail(ctx, FESC_ELEVEL, "linear: level out of range");
    for (uint32_t q = 1; q < n1; q++)
        if (!ctx->keys.count(desc->baby_key_base + q))
            return fesc_fail(ctx, FESC_ENOKEY, "linear: missing baby-step key " + std::to_string(desc->baby_key_base + q));
    for (uint32_t p = 1; p < n2; p++)
        if (!ctx->keys.count(desc->giant_key_base + p))
            return fesc_fail(ctx, FESC_ENOKEY, "linear: missing giant-step key " + std::to_string(desc->giant_key_base + p));
    cudaStream_t st = (cudaStream_t)stream;
    const size_t ctw = (size_t)2 * level * N;
    // token blocks per group, from the scratch budget
    const size_t per_tb = ((size_t)gin * n1 + (size_t)nout * n2) * ctw * sizeof(u64);
    uint32_t tbg = (uint32_t)(bsgs_group_bytes(ctx) / per_tb);
    if (tbg < 1) tbg = 1;
    if (tbg > tbs) tbg = tbs;
    const uint32_t max_batch = tbg * (gin > nout ? gin : nout);
    const size_t ks_words = ks_scratch_words(ctx, level, ks_chunk(ctx, max_batch));
    const size_t rs_words = (size_t)(tbg * nout < 16384 ? tbg * nout : 16384) * 2 * N;
    const size_t rot_words = (size_t)tbg * gin * n1 * ctw, acc_words = (size_t)tbg * nout * n2 * ctw;
    u64* scratch;
    int rc = ctx_scratch(ctx, (rot_words + acc_words + (ks_words > rs_words ? ks_words : rs_words)) * sizeof(u64), &scratch);
    if (rc != FESC_OK) return rc;
    u64* rot = scratch;
    u64* acc = rot + rot_words;
    u64* ks = acc + acc_words;
    // lazy 128-bit sums: reduce before terms * q^2 could reach 2^128
    uint32_t qbits = 0;
    for (uint32_t i = 0; i < level; i++) {
        uint32_t b = 64 - __builtin_clzll(ctx->q[i]);
        if (b > qbits) qbits = b;
    }
    uint32_t reduce_every = 2 * qbits >= 127 ? 1 : (2 * qbits <= 96 ? 0x7fffffffu : (1u << (127 - 2 * qbits)));
    const u64* in = (const u64*)d_ct_in;
    const u64* diags = (const u64*)d_diags;
    u64* out = (u64*)d_ct_out;
    for (uint32_t tb0 = 0; tb0 < tbs; tb0 += tbg) {
        const uint32_t nt = tbs - tb0 < tbg ? tbs - tb0 : tbg;
        const u64* gin_base = in + (size_t)tb0 * gin * ctw;
        // slot q = 0 of the rotated set is the input itself
        FESC_CHECK_CUDA(ctx, cudaMemcpy2DAsync(rot, (size_t)n1 * ctw * sizeof(u64), gin_base, ctw * sizeof(u64),
                                               ctw * sizeof(u64), (size_t)nt * gin, cudaMemcpyDeviceToDevice, st));
        if (desc->hoist && n1 > 1) {
            std::vector<uint32_t> ids;
            for (uint32_t q = 1; q < n1; q++) ids.push_back(desc->baby_key_base + q);
            rc = rotate_hoisted_internal(ctx, gin_base, ctw, rot + ctw, (size_t)n1 * ctw, ctw, nt * gin, level, ids.data(),
                                         n1 - 1, ks, st);
            if (rc != FESC_OK) return rc;
        } else {
            for (uint32_t q = 1; q < n1; q++) {
                rc = rotate_internal(ctx, gin_base, ctw, rot + (size_t)q * ctw, (size_t)n1 * ctw, nt * gin, level,
                                     desc->baby_key_base + q, ks, st, 0);
                if (rc != FESC_OK) return rc;
            }
        }
        const uint32_t bp_count = nout * n2;
        prof_begin(ctx, PF_BSGS, st);
#define BSGS(TT, PT)                                                                                          \
    do {                                                                                                      \
        dim3 grid((bp_count + PT - 1) / PT, (N + 255) / 256, level * ((nt + TT - 1) / TT));                   \
        if (grid.z > 65535) return fesc_fail(ctx, FESC_EINVAL, "linear: too many accumulator tiles");         \
        k_bsgs_accumulate<TT, PT><<<grid, 256, 0, st>>>(rot, diags, acc, ctx->d_pc, N, level, nt, gin * n1,  \
                                                        bp_count, reduce_every);                              \
    } while (0)
#define BSGS_FP(TT, PT)                                                                                       \
    do {                                                                                                      \
        dim3 grid((bp_count + PT - 1) / PT, (N + 255) / 256, level * ((nt + TT - 1) / TT));                   \
        if (grid.z > 65535) return fesc_fail(ctx, FESC_EINVAL, "linear: too many accumulator tiles");         \
        k_bsgs_accumulate_fp<TT, PT><<<grid, 256, 0, st>>>(rot, diags, acc, ctx->d_pc, N, level, nt, gin * n1, \
                                                           bp_count);                                         \
    } while (0)
#define BSGS_FPS(TT, PT, ST)                                                                                  \
    do {                                                                                                      \
        dim3 grid((bp_count + PT - 1) / PT, N / 256, level * ((nt + TT - 1) / TT));                           \
        if (grid.z > 65535) return fesc_fail(ctx, FESC_EINVAL, "linear: too many accumulator tiles");         \
        const size_t smem = (size_t)ST * (2 * TT + PT) * 2048;                                                \
        auto kern = k_bsgs_accumulate_fp_staged<TT, PT, ST>;                                                  \
        FESC_CHECK_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        kern<<<grid, 256, smem, st>>>(rot, diags, acc, ctx->d_pc, N, level, nt, gin * n1, bp_count);          \
    } while (0)
        // all active primes below 2^50: exact FP64 products (staged variant when rows split into 256-word tiles);
        // otherwise 128-bit integer accumulation.  FESC_BSGS_INT=1 forces the integer kernel (for comparisons).
#define BSGS_MIX(TT, PT, ST)                                                                                  \
    do {                                                                                                      \
        dim3 grid(((bp_count + PT - 1) / PT) * ((nt + TT - 1) / TT), N / MIX_THREADS, level);                 \
        const size_t smem = (size_t)ST * (2 * TT + PT) * MIX_THREADS * 8;                                     \
        auto kern = k_bsgs_accumulate_mixed<TT, PT, ST>;                                                      \
        FESC_CHECK_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        kern<<<grid, MIX_THREADS, smem, st>>>(rot, diags, acc, ctx->d_pc, N, level, nt, gin * n1, bp_count);  \
    } while (0)
        const bool fp_ok = qbits <= 50 && bsgs_kernel() != 2;
        if (fp_ok && bsgs_kernel() == 0 && N % 256 == 0 && nt >= 2 && gin * n1 <= 256) BSGS_MIX(2, 8, 3);
        else if (fp_ok && N % 256 == 0 && nt >= 2) BSGS_FPS(2, 8, 3);
        else if (fp_ok && nt >= 2) BSGS_FP(2, 8);
        else if (fp_ok) BSGS_FP(1, 8);
        else if (nt >= 2) BSGS(2, 8);
        else BSGS(1, 8);
#undef BSGS
        prof_end(ctx, PF_BSGS, st);
        FESC_CHECK_CUDA(ctx, cudaGetLastError());
        ctx->counters[2] += (uint64_t)nt * bp_count * gin * n1;
        if (desc->defer) {
            rc = giant_sum_deferred_internal(ctx, acc, n2, ctw, nt * nout, level, desc->giant_key_base, ks, st);
            if (rc != FESC_OK) return rc;
        } else {
            for (uint32_t p = 1; p < n2; p++) {
                rc = rotate_internal(ctx, acc + (size_t)p * ctw, (size_t)n2 * ctw, acc, (size_t)n2 * ctw, nt * nout,
                                     level, desc->giant_key_base + p, ks, st, 1);
                if (rc != FESC_OK) return rc;
            }
        }
        rc = rescale_internal(ctx, acc, (size_t)n2 * ctw, out + (size_t)tb0 * nout * 2 * (level - 1) * N, nt * nout, level,
                              ks, st);
        if (rc != FESC_OK) return rc;
    }
    return FESC_OK;
}
