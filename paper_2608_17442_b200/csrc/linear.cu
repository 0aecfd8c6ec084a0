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

#define FESC_DBG_FILE 4   // file id in the sites a debug build reports
#include "ops.cuh"

// Debug build: the spans an accumulate CTA reads and writes (token blocks [tb0, tb0 + tt), (b,p) pairs [bp0, bp0 + pt),
// all terms, both polynomials, every limb), the same for all its threads.
__device__ __forceinline__ bool dbg_accumulate_spans(const u64* rot, const u64* diags, const u64* acc, uint32_t N, uint32_t level,
                                                     uint32_t tbs, uint32_t terms, uint32_t bp_count, uint32_t tb0,
                                                     uint32_t bp0, uint32_t tt, uint32_t pt) {
#ifdef FESC_DEBUG_BOUNDS
    const size_t poly = (size_t)level * N, ctw = 2 * poly;
    for (uint32_t i = 0; i < tt && tb0 + i < tbs; i++) {
        if (!DBG_REGION(rot + (size_t)(tb0 + i) * terms * ctw, terms * ctw * sizeof(u64))) return false;
        for (uint32_t j = 0; j < pt && bp0 + j < bp_count; j++)
            if (!DBG_REGION(acc + ((size_t)(tb0 + i) * bp_count + bp0 + j) * ctw, ctw * sizeof(u64))) return false;
    }
    for (uint32_t j = 0; j < pt && bp0 + j < bp_count; j++)
        if (!DBG_REGION(diags + (size_t)(bp0 + j) * terms * poly, terms * poly * sizeof(u64))) return false;
#endif
    return true;
}

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
    if (!dbg_accumulate_spans(rot, diags, acc, N, level, tbs, terms, bp_count, tb0, bp0, TT, PT)) return;
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
    if (!dbg_accumulate_spans(rot, diags, acc, N, level, tbs, terms, bp_count, tb0, bp0, TT, PT)) return;
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
    if (!dbg_accumulate_spans(rot, diags, acc, N, level, tbs, terms, bp_count, tb0, bp0, TT, PT)) return;   // before any barrier
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
    if (!dbg_accumulate_spans(rot, diags, acc, N, level, tbs, terms, bp_count, tb0, bp0, TT, PT)) return;   // before any barrier
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

// Tensor-core accumulate for primes below 2^56 (at most 256 terms).  For one coefficient of one limb the sums
//   S[tb,p][bp] = sum_t x_t[tb,p] * w_t[bp]
// are a small dense integer matrix product over the terms.  Every residue is cut into 7 bytes; the byte planes
// form u8 matrices and  S = sum_{k,j} 256^(k+j) D[k][j],  D[k][j] = sum_t w_t.byte(k) * x_t.byte(j),  where each
// D is an exact s32 accumulator of mma.sync m16n8k32 (u8 x u8): 256 terms of 255^2 stay below 2^24.
// Mapping: a warp owns ONE coefficient; M side = 8 (b,p) outputs x 2 byte planes per 16-row tile (4 tiles, the
// last one half empty), N side = 8 (token block, polynomial) columns x 1 byte plane per 8-column tile (7 tiles),
// K = 32 terms per instruction.  With that mapping lane (g, tg) ends up holding all 49 byte-plane sums of output
// bp = g for token block tg and both polynomials, so the recombination needs no exchange between lanes.
// A CTA = 8 warps = 8 neighbouring coefficients of one limb, 4 token blocks and ALL (b,p) outputs: the rotated
// inputs of its coefficients stay in shared memory for the whole CTA, the diagonals stream through an 8-stage
// cp.async ring (4 stages when more than 128 terms leave less room) (32 terms x 8 outputs x 8 coefficients per stage), every operand word is read from HBM once per
// launch.  Fragments are built in registers from the raw 64-bit words: four words of consecutive terms are
// byte-transposed with 15 byte permutes into the seven 4-term registers the instruction expects.
// Recombination: E_d = sum_{k+j=d} D[k][j] (13 values below 2^27), groups of four E_d are packed exactly into
// doubles T_m < 2^52, and S mod q = T_0 + T_1 2^32 + T_2 2^64 + T_3 2^96 mod q with exact FP64 products (primes below
// 2^50) or as a 128-bit integer followed by the usual reduction (primes of 50..55 bits).
#define IM_CW 8
#define IM_ROWP 9                      // words per (row, 8 coefficients): one word of padding
#define IM_BPP (32 * IM_ROWP + 1)      // words between the (b,p) blocks of a stage (= 1 mod 16: conflict-free fragment loads)
#define IM_STAGE_WORDS (8 * IM_BPP)

__device__ __forceinline__ void cp_async8z(uint32_t smem_dst, const void* gmem_src, bool valid) {
    const uint32_t n = valid ? 8u : 0u;      // 0 source bytes: the destination is filled with zeros
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(smem_dst), "l"(gmem_src), "r"(n) : "memory");
}

template <bool FP, int IM_STAGES>
__global__ void __launch_bounds__(32 * IM_CW, 1) k_bsgs_accumulate_imma(
    const u64* __restrict__ rot, const u64* __restrict__ diags, u64* __restrict__ acc,
    const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level, uint32_t tbs, uint32_t terms, uint32_t bp_count,
    uint32_t xs_pitch) {
    extern __shared__ __align__(16) u64 stage[];      // x: [8 (tb,p)][xs_pitch], then IM_STAGES x [8 (b,p)][IM_BPP]
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tg = lane & 3;
    const uint32_t c0 = blockIdx.x * IM_CW, l = blockIdx.y, tb0 = blockIdx.z * 4;
    if (!dbg_accumulate_spans(rot, diags, acc, N, level, tbs, terms, bp_count, tb0, 0, 4, bp_count)) return;   // before any barrier
    const PrimeConst pc = pcs[l];
    const size_t poly = (size_t)level * N, ctw = 2 * poly;
    const uint32_t ksteps = (terms + 31) >> 5, bp_tiles = (bp_count + 7) >> 3, total = ksteps * bp_tiles;
    const uint32_t sm_base = (uint32_t)__cvta_generic_to_shared(stage);
    const uint32_t cw = tid & 7, rw = tid >> 3;       // word of a row, row of a pass (32 rows per pass)
    const size_t goff = (size_t)l * N + c0 + cw;
    // rotated inputs of the CTA's coefficients: rows (tb,p) x terms, zero beyond `terms`
    {
        const uint32_t tp = ksteps << 5;
#pragma unroll 1
        for (uint32_t tbp = 0; tbp < 8; tbp++) {
            const uint32_t tb = tb0 + (tbp >> 1) < tbs ? tb0 + (tbp >> 1) : tbs - 1;
            const u64* src = rot + goff + (size_t)tb * terms * ctw + (tbp & 1) * poly + (size_t)rw * ctw;
            uint32_t dst = sm_base + (tbp * xs_pitch + rw * IM_ROWP + cw) * 8;
#pragma unroll 1
            for (uint32_t t = rw; t < tp; t += 32) {
                cp_async8z(dst, t < terms ? src : rot, t < terms);
                src += 32 * ctw;
                dst += 32 * IM_ROWP * 8;
            }
        }
        cp_async_commit();
    }
    // diagonals: a ring of stages, one stage = 32 terms x 8 outputs; this thread copies word cw of term rw of each output
    const size_t bp_stride = (size_t)terms * poly;
    const u64* ld_src = diags + goff + (size_t)rw * poly;     // output 0 of the tile to request, term rw of its k-step
    uint32_t ld_ks = 0, ld_left = bp_count;                   // outputs from the requested tile on
    uint32_t ld_dst = sm_base + (8 * xs_pitch + rw * IM_ROWP + cw) * 8;
    const uint32_t ring_end = sm_base + (8 * xs_pitch + IM_STAGES * IM_STAGE_WORDS) * 8;
    auto issue = [&]() {
        const bool valid = (ld_ks << 5) + rw < terms;
        const u64* src = valid ? ld_src : diags;
        const uint32_t last = ld_left < 8 ? ld_left - 1 : 7;   // a partial tile repeats its last output
#pragma unroll
        for (uint32_t i = 0; i < 8; i++) cp_async8z(ld_dst + i * (IM_BPP * 8), src + (i < last ? i : last) * bp_stride, valid);
        ld_src += 32 * poly;
        if (++ld_ks == ksteps) {
            ld_ks = 0;
            ld_src += 8 * bp_stride - (size_t)ksteps * 32 * poly;
            ld_left -= 8;
        }
        ld_dst += IM_STAGE_WORDS * 8;
        if (ld_dst >= ring_end) ld_dst -= IM_STAGES * IM_STAGE_WORDS * 8;
    };
    for (uint32_t s = 0; s < IM_STAGES - 1; s++) {
        if (s < total) issue();
        cp_async_commit();
    }
    // constants of the recombination
    const double q = pc.qd, qinv = pc.qinvd;
    double c32 = 0, c64 = 0, c96 = 0;
    if (FP) {
        c32 = fp_reduce(4294967296.0, q, qinv);
        c64 = fp_modmul(c32, c32, q, qinv);
        c96 = fp_modmul(c64, c32, q, qinv);
    }
    int d[4][7][4];
    int z0 = 0, z1 = 0, z2 = 0, z3 = 0;       // a fixed quad of zero addends (see imma_u8_zero)
    asm volatile("" : "+r"(z0), "+r"(z1), "+r"(z2), "+r"(z3));
    const u64* a_ring = stage + 8 * xs_pitch + g * IM_BPP + (4 * tg) * IM_ROWP + warp;
    const u64* b_frag = stage + g * xs_pitch + (4 * tg) * IM_ROWP + warp;
    uint32_t slot = 0, s = 0;
#pragma unroll 1
    for (uint32_t bt = 0; bt < bp_tiles; bt++) {
#pragma unroll 1
        for (uint32_t ks = 0; ks < ksteps; ks++, s++) {
            cp_async_wait<IM_STAGES - 2>();
            __syncthreads();                  // stage s has landed for everyone; the slot of stage s-1 is free
            if (s + IM_STAGES - 1 < total) issue();
            cp_async_commit();
            uint32_t fa[2][7], fb[2][7];
            const u64* A = a_ring + slot * IM_STAGE_WORDS;
            const u64* X = b_frag + (ks << 5) * IM_ROWP;
#pragma unroll
            for (int h = 0; h < 2; h++) {
                byte_planes4(A[(16 * h) * IM_ROWP], A[(16 * h + 1) * IM_ROWP], A[(16 * h + 2) * IM_ROWP],
                             A[(16 * h + 3) * IM_ROWP], fa[h]);
                byte_planes4(X[(16 * h) * IM_ROWP], X[(16 * h + 1) * IM_ROWP], X[(16 * h + 2) * IM_ROWP],
                             X[(16 * h + 3) * IM_ROWP], fb[h]);
            }
            slot = slot + 1 == IM_STAGES ? 0 : slot + 1;
            if (ks == 0) {                    // the first k-step of a tile starts from zero accumulators
#pragma unroll
                for (int m = 0; m < 4; m++)
#pragma unroll
                    for (int j = 0; j < 7; j++)
                        imma_u8_zero(d[m][j], fa[0][2 * m], m < 3 ? fa[0][2 * m + 1] : 0u, fa[1][2 * m],
                                     m < 3 ? fa[1][2 * m + 1] : 0u, fb[0][j], fb[1][j], z0, z1, z2, z3);
            } else {
#pragma unroll
                for (int m = 0; m < 4; m++)
#pragma unroll
                    for (int j = 0; j < 7; j++)
                        imma_u8(d[m][j], fa[0][2 * m], m < 3 ? fa[0][2 * m + 1] : 0u, fa[1][2 * m],
                                m < 3 ? fa[1][2 * m + 1] : 0u, fb[0][j], fb[1][j]);
            }
        }
        // recombine: lane (g, tg) holds output bp = 8 bt + g of token block tb0 + tg, both polynomials
        const uint32_t bp = bt * 8 + g, tb = tb0 + tg;
        const bool live = bp < bp_count && tb < tbs;
        u64* dst = acc + ((size_t)(live ? tb : 0) * bp_count + (live ? bp : 0)) * ctw + (size_t)l * N + c0 + warp;
        if (live) {
            dst[0] = imma_recombine<FP>(d, 0, pc, c32, c64, c96);
            dst[poly] = imma_recombine<FP>(d, 1, pc, c32, c64, c96);
        }
    }
    cp_async_wait<0>();
}

// Knobs for experiments.  FESC_BSGS_KERNEL picks the accumulate kernel: "int" the 128-bit integer one, "fp" the
// exact-FP64 one, "mixed" the mixed-pipe one, anything else the default (tensor-core byte planes where they apply).  FESC_BSGS_GROUP_GIB fixes the scratch
// budget that decides how many token blocks are processed per group (default: from the free device memory).
static int bsgs_kernel() {
    static int v = -1;
    if (v < 0) {
        const char* e = getenv("FESC_BSGS_KERNEL");
        v = !e ? 0 : (!strcmp(e, "int") ? 2 : (!strcmp(e, "fp") ? 1 : (!strcmp(e, "mixed") ? 3 : 0)));
    }
    return v;
}
// Larger groups re-read the diagonals less often and give the key-switch kernels larger batches; every token block
// of a group needs its rotated inputs and its partial sums resident.  Budget: 28 GiB of scratch for them (37 GiB with packed operands, whose packed inputs
// and key-switch chunk count as well; 44 GiB allows groups of 8; a fixed figure, so the launch shape does not depend on what else holds memory); if the device cannot provide the scratch,
// the group is halved until it fits.
static size_t bsgs_group_bytes(bool packed) {
    const char* e = getenv("FESC_BSGS_GROUP_GIB");
    if (e && atoi(e) > 0) return (size_t)atoi(e) << 30;
    return (size_t)(packed ? 37 : 28) << 30;
}

// Projection on packed diagonals.  Token blocks are processed in groups of up to 8 = two tiles of 4: the baby rotations
// run on 4 token blocks at a time and their results are packed into the group's fragment images; the accumulate then
// covers both tiles in one launch (the two CTAs that need the same diagonal images run side by side, so the images
// cross HBM once per group), for one part of the output blocks at a time so that the partial sums of a part stay
// small; giant steps and rescale follow per part.  With groups of 8 the image is streamed twice per 16 token blocks
// instead of four times.
static int linear_packed(fesc_ctx* ctx, const u64* in, const uint8_t* image, const fesc_bsgs_desc* desc, u64* out,
                         cudaStream_t st, uint32_t qbits) {
    const uint32_t n1 = desc->n1, n2 = desc->n2, gin = desc->in_blocks, nout = desc->out_blocks;
    const uint32_t tbs = desc->token_blocks, level = desc->n_limbs, N = ctx->N, terms = gin * n1;
    const size_t ctw = (size_t)2 * level * N, ctw_out = (size_t)2 * (level - 1) * N;
    uint32_t bstep = 8;                    // a part starts at a (b,p) pair that is a multiple of 8
    while (bstep > 1 && (bstep / 2) * n2 % 8 == 0) bstep /= 2;
    if (n2 % 8 == 0) bstep = 1;
    u64 *scratch = nullptr, *rot = nullptr, *acc = nullptr, *ks = nullptr;
    uint8_t* xpk = nullptr;
    uint32_t tbg = tbs >= 8 ? 8 : tbs, nb_part = nout;
    int rc = FESC_ENOMEM;
    for (;; tbg = tbg > 4 ? 4 : (tbg + 1) / 2) {
        const uint32_t parts = (tbg + 3) / 4, sub = tbg < 4 ? tbg : 4;
        nb_part = (nout + parts - 1) / parts;
        nb_part = (nb_part + bstep - 1) / bstep * bstep;
        if (nb_part > nout) nb_part = nout;
        const uint32_t max_batch = sub * gin > tbg * nb_part ? sub * gin : tbg * nb_part;
        const size_t ks_words = ks_scratch_words(ctx, level, ks_chunk(ctx, max_batch), desc->defer ? giant_ext_buffers(n2) : 1);
        const size_t rs_words = (size_t)(nb_part < 16384 ? nb_part : 16384) * 2 * N;
        const size_t rot_words = (size_t)sub * terms * ctw, acc_words = (size_t)tbg * nb_part * n2 * ctw;
        const size_t xpk_words = bsgs_packed_bytes(N, level, 2 * tbg, terms) / 8;
        const size_t total = (rot_words + acc_words + xpk_words + (ks_words > rs_words ? ks_words : rs_words)) * sizeof(u64);
        if (total <= bsgs_group_bytes(true) || tbg == 1) {
            rc = ctx_scratch(ctx, total, &scratch);
            if (rc == FESC_OK) {
                rot = scratch;
                acc = rot + rot_words;
                xpk = (uint8_t*)(acc + acc_words);
                ks = acc + acc_words + xpk_words;
                break;
            }
            if (rc != FESC_ENOMEM) return rc;
        }
        if (tbg == 1) return rc;
    }
    ctx->counters[5] = tbg;
    const size_t tile_bytes = bsgs_packed_bytes(N, level, 8, terms);     // one tile of 8 rows of packed inputs
    const uint32_t dshift = desc->diag_run_log2;
    const size_t image_tile_bytes = bsgs_packed_bytes(N >> dshift, level, 8, terms);
    for (uint32_t tb0 = 0; tb0 < tbs; tb0 += tbg) {
        const uint32_t nt = tbs - tb0 < tbg ? tbs - tb0 : tbg;
        for (uint32_t s0 = 0; s0 < nt; s0 += 4) {        // baby rotations of 4 token blocks, packed into their tile
            const uint32_t ns = nt - s0 < 4 ? nt - s0 : 4;
            const u64* gin_base = in + (size_t)(tb0 + s0) * gin * ctw;
            FESC_CHECK_CUDA(ctx, cudaMemcpy2DAsync(rot, (size_t)n1 * ctw * sizeof(u64), gin_base, ctw * sizeof(u64),
                                                   ctw * sizeof(u64), (size_t)ns * gin, cudaMemcpyDeviceToDevice, st));
            if (desc->hoist && n1 > 1) {
                std::vector<uint32_t> ids;
                for (uint32_t q = 1; q < n1; q++) ids.push_back(desc->baby_key_base + q);
                rc = rotate_hoisted_internal(ctx, gin_base, ctw, rot + ctw, (size_t)n1 * ctw, ctw, ns * gin, level, ids.data(),
                                             n1 - 1, ks, st);
                if (rc != FESC_OK) return rc;
            } else {
                for (uint32_t q = 1; q < n1; q++) {
                    rc = rotate_internal(ctx, gin_base, ctw, rot + (size_t)q * ctw, (size_t)n1 * ctw, ns * gin, level,
                                         desc->baby_key_base + q, ks, st, 0);
                    if (rc != FESC_OK) return rc;
                }
            }
            if ((rc = bsgs_pack_inputs(ctx, rot, xpk + (size_t)(s0 / 4) * tile_bytes, level, ns, terms, st)) != FESC_OK) return rc;
        }
        for (uint32_t b0 = 0; b0 < nout; b0 += nb_part) {
            const uint32_t nb = nout - b0 < nb_part ? nout - b0 : nb_part;
            rc = bsgs_accumulate_packed(ctx, xpk, image + (size_t)(b0 * n2 / 8) * image_tile_bytes, acc, level, nt, terms, nb * n2,
                                        qbits <= 50, dshift, st);
            if (rc != FESC_OK) return rc;
            ctx->counters[2] += (uint64_t)nt * nb * n2 * terms;
            if (desc->defer) {
                rc = giant_sum_deferred_internal(ctx, acc, n2, ctw, nt * nb, level, desc->giant_key_base, ks, st);
                if (rc != FESC_OK) return rc;
            } else {
                for (uint32_t p = 1; p < n2; p++) {
                    rc = rotate_internal(ctx, acc + (size_t)p * ctw, (size_t)n2 * ctw, acc, (size_t)n2 * ctw, nt * nb, level,
                                         desc->giant_key_base + p, ks, st, 1);
                    if (rc != FESC_OK) return rc;
                }
            }
            for (uint32_t tb = 0; tb < nt; tb++) {      // the outputs of a token block are contiguous, those of a part are not
                rc = rescale_internal(ctx, acc + (size_t)tb * nb * n2 * ctw, (size_t)n2 * ctw,
                                      out + ((size_t)(tb0 + tb) * nout + b0) * ctw_out, nb, level, ks, st);
                if (rc != FESC_OK) return rc;
            }
        }
    }
    return FESC_OK;
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
    const bool packed = desc->packed != 0;
    if (!packed && desc->diag_run_log2)
        return fesc_fail(ctx, FESC_EINVAL, "linear: periodic diagonals (diag_run_log2) are a property of the packed image");
    if (packed && !bsgs_packed_supported(ctx, level, gin * n1, desc->diag_run_log2))
        return fesc_fail(ctx, FESC_EINVAL, "linear: packed diagonals need N a multiple of 8, primes below 2^56, at most 512 terms and runs that leave 8 words per limb");
    if (packed) {
        uint32_t bits = 0;
        for (uint32_t i = 0; i < level; i++) {
            const uint32_t b = 64 - __builtin_clzll(ctx->q[i]);
            if (b > bits) bits = b;
        }
        return linear_packed(ctx, (const u64*)d_ct_in, (const uint8_t*)d_diags, desc, (u64*)d_ct_out, st, bits);
    }
    // residue diagonals from here on; token blocks per group, from the scratch budget
    const size_t per_tb = ((size_t)gin * n1 + (size_t)nout * n2) * ctw * sizeof(u64);
    uint32_t tbg = (uint32_t)(bsgs_group_bytes(false) / per_tb);
    if (tbg < 1) tbg = 1;
    if (tbg > tbs) tbg = tbs;
    u64 *scratch = nullptr, *rot = nullptr, *acc = nullptr, *ks = nullptr;
    int rc;
    for (;;) {
        const uint32_t max_batch = tbg * (gin > nout ? gin : nout);
        const size_t ks_words = ks_scratch_words(ctx, level, ks_chunk(ctx, max_batch), desc->defer ? giant_ext_buffers(n2) : 1);
        const size_t rs_words = (size_t)(tbg * nout < 16384 ? tbg * nout : 16384) * 2 * N;
        const size_t rot_words = (size_t)tbg * gin * n1 * ctw, acc_words = (size_t)tbg * nout * n2 * ctw;
        rc = ctx_scratch(ctx, (rot_words + acc_words + (ks_words > rs_words ? ks_words : rs_words)) * sizeof(u64), &scratch);
        if (rc == FESC_OK) {
            rot = scratch;
            acc = rot + rot_words;
            ks = acc + acc_words;
            break;
        }
        if (rc != FESC_ENOMEM || tbg == 1) return rc;
        tbg = (tbg + 1) / 2;
    }
    ctx->counters[5] = tbg;
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
#define BSGS_IMMA(FP, ST)                                                                                       \
    do {                                                                                                      \
        const uint32_t tp = ((gin * n1 + 31) / 32) * 32;                                                      \
        uint32_t pitch = tp * IM_ROWP;                                                                        \
        pitch += (17 - pitch % 16) % 16;          /* = 1 mod 16 */                                            \
        dim3 grid(N / IM_CW, level, (nt + 3) / 4);                                                            \
        const size_t smem = ((size_t)8 * pitch + (size_t)ST * IM_STAGE_WORDS) * 8;                            \
        auto kern = k_bsgs_accumulate_imma<FP, ST>;                                                           \
        FESC_CHECK_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        kern<<<grid, 32 * IM_CW, smem, st>>>(rot, diags, acc, ctx->d_pc, N, level, nt, gin * n1, bp_count, pitch); \
    } while (0)
        const bool fp_ok = qbits <= 50 && bsgs_kernel() != 2;
        const bool imma_ok = bsgs_kernel() == 0 && qbits <= 56 && N % IM_CW == 0 && gin * n1 <= 256 && level <= 65535;
        const bool deep = gin * n1 <= 128;       // room for 8 stages beside the rotated inputs
        if (imma_ok && qbits <= 50 && deep) BSGS_IMMA(true, 8);
        else if (imma_ok && qbits <= 50) BSGS_IMMA(true, 4);
        else if (imma_ok && deep) BSGS_IMMA(false, 8);
        else if (imma_ok) BSGS_IMMA(false, 4);
        else if (fp_ok && bsgs_kernel() == 3 && N % 256 == 0 && nt >= 2 && gin * n1 <= 256) BSGS_MIX(2, 8, 3);
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
