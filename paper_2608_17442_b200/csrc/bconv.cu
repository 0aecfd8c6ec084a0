// Fast basis conversion of the division by P (special-prime residues -> data primes) on the tensor cores.
//
// The conversion is, per coefficient, a small dense integer matrix product  out_t = sum_k y_k * M[k][t] (mod q_t)
// with at most 4 source residues y_k and up to 32 target moduli.  Written on byte planes,
//     out_t = sum_a 256^a  sum_{k,b} C[t][k][b].byte(a) * y_k.byte(b),     C[t][k][b] = M[k][t] * 256^b mod q_t,
// the inner sum is exactly one u8 x u8 -> s32 m16n8k32 tensor instruction per plane a and tile of 16 targets: the K
// dimension is (4 sources) x (8 bytes of a 64-bit word), so a source word goes into the B operand as it is, without any
// byte transposition; the A operands are constants (fragment images built on the host with the tables).  Every sum is
// below 32 * 255^2 < 2^21, the planes recombine into lo + 2^32 hi (both below 2^47), and one exact FP64 product (targets
// below 2^50) or one 128-bit reduction (larger targets) gives the residue: about 16 instructions per output instead of
// four modular products.  Results are the canonical residues (or the centred doubles the forward transform takes), bit
// for bit those of the scalar kernel in ops.cu, which remains for the shapes this one does not cover.  (The same scheme
// for the ModUp of a key-switch digit was measured and dropped: 76 ms per projection step against 52 ms for the scalar
// kernel, whose four exact FP64 products per output cost about what the recombination of eight planes costs.)
#define FESC_DBG_FILE 10   // file id in the sites a debug build reports
#include "ops.cuh"

#define BC_WARPS 4
#ifndef BC_MINB
#define BC_MINB 4
#endif
#ifndef BC_UNROLL
#define BC_UNROLL 1
#endif
#define BC_PRAGMA(x) _Pragma(#x)
#define BC_UNROLL_N(n) BC_PRAGMA(unroll n)
#define BC_COEFS 64        // coefficients per warp: 8 groups of 8
#define BC_FRAG_WORDS (2 * 8 * 32)   // uint4 per conversion: [tile][plane][lane]

// This lane's source word y belongs to source k = lane & 3 and coefficient g = lane >> 2 of the group.  lo / hi of the
// lane's outputs: r = 0, 1: target row 16 t + g, coefficients 2 tg, 2 tg + 1; r = 2, 3: target row 16 t + g + 8.
template <int TILES>
__device__ __forceinline__ void bconv_mma(u64 y, const uint4* __restrict__ sfrag, uint32_t lane, u64 (&lo)[TILES][4],
                                          u64 (&hi)[TILES][4], int z0, int z1, int z2, int z3) {
    const uint32_t tg = lane & 3, src0 = (lane & ~3u) | (tg >> 1), src1 = src0 + 2;
    const uint32_t ylo = (uint32_t)y, yhi = (uint32_t)(y >> 32);
    const uint32_t l0 = __shfl_sync(0xffffffffu, ylo, src0), h0 = __shfl_sync(0xffffffffu, yhi, src0);
    const uint32_t l1 = __shfl_sync(0xffffffffu, ylo, src1), h1 = __shfl_sync(0xffffffffu, yhi, src1);
    // K index = 8 k + b: bytes 4 tg .. 4 tg + 3 are one half of source tg >> 1, bytes 16 + 4 tg .. of source 2 + (tg >> 1)
    const uint32_t b0 = (tg & 1) ? h0 : l0, b1 = (tg & 1) ? h1 : l1;
#pragma unroll
    for (int t = 0; t < TILES; t++) {
        int d[8][4];
#pragma unroll
        for (int a = 0; a < 8; a++) {
            const uint4 A = sfrag[(t * 8 + a) * 32 + lane];
            imma_u8_zero(d[a], A.x, A.y, A.z, A.w, b0, b1, z0, z1, z2, z3);
        }
#pragma unroll
        for (int r = 0; r < 4; r++) {       // every plane sum is below 2^21: pairs fit 32 bits, fours 64 bits
            const uint32_t t01 = (uint32_t)d[0][r] + ((uint32_t)d[1][r] << 8), t23 = (uint32_t)d[2][r] + ((uint32_t)d[3][r] << 8);
            const uint32_t t45 = (uint32_t)d[4][r] + ((uint32_t)d[5][r] << 8), t67 = (uint32_t)d[6][r] + ((uint32_t)d[7][r] << 8);
            lo[t][r] = (u64)t01 + ((u64)t23 << 16);
            hi[t][r] = (u64)t45 + ((u64)t67 << 16);
        }
    }
}
// lo + 2^32 hi modulo a prime below 2^50, as an exact double with magnitude below 2^47 + q
__device__ __forceinline__ double bconv_fp(u64 lo, u64 hi, double c32, double q, double qinv) {
    return fp_from_u64(lo) + fp_modmul(fp_from_u64(hi), c32, q, qinv);
}
__device__ __forceinline__ u64 bconv_int(u64 lo, u64 hi, const PrimeConst& pc) {
    const u128 S = ((u128)hi << 32) + lo;
    return reduce128((u64)(S >> 64), (u64)S, pc);
}

// ---------------------------------------------------------------------------------------
// Division by P, conversion step: u[bp][i] = sum_k y_k ((P/p_k) mod q_i) - #{y_k > p_k/2} P,  y_k = r_k (P/p_k)^-1 mod p_k.
// grid = (N / 256, polynomials), 4 warps x 64 coefficients.
// ---------------------------------------------------------------------------------------
template <int TILES>
__global__ void __launch_bounds__(32 * BC_WARPS, BC_MINB) k_moddown_conv_imma(const u64* __restrict__ acc, u64* __restrict__ u,
                                                                     const ModDownTab* __restrict__ tab, const uint4* __restrict__ frag,
                                                                     const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level,
                                                                     uint32_t n_q, uint32_t K, int out_double) {
    __shared__ uint4 sfrag[BC_FRAG_WORDS];
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tg = lane & 3;
    const uint32_t bp = blockIdx.y, rows = level + K;
    if (!DBG_REGION(acc + ((size_t)bp * rows + level) * N, (size_t)K * N * sizeof(u64)) ||
        !DBG_REGION(u + (size_t)bp * level * N, (size_t)level * N * sizeof(u64)) || !DBG_REGION(tab, sizeof(ModDownTab)))
        return;                                     // the same for every thread of the CTA (a barrier follows)
    for (uint32_t i = tid; i < TILES * 8 * 32; i += 32 * BC_WARPS) sfrag[i] = frag[i];
    __syncthreads();
    const bool has = tg < K;
    u64 inv = 0, invs = 0, pk = 1, half = 0;
    if (has) inv = tab->inv[tg], invs = tab->invs[tg], pk = pcs[n_q + tg].q, half = tab->half[tg];
    const u64* src = acc + ((size_t)bp * rows + level + (has ? tg : 0)) * N + g;
    u64* out = u + (size_t)bp * level * N + 2 * tg;
    int z0 = 0, z1 = 0, z2 = 0, z3 = 0;
    asm volatile("" : "+r"(z0), "+r"(z1), "+r"(z2), "+r"(z3));
    const uint32_t c_base = (blockIdx.x * BC_WARPS + warp) * BC_COEFS;
    u64 raw[BC_COEFS / 8];                      // the warp's source words, all requested before the first is used
#pragma unroll
    for (int grp = 0; grp < BC_COEFS / 8; grp++) raw[grp] = has ? src[c_base + grp * 8] : 0;
    bool live[TILES][2], fp[TILES][2];          // the rows this lane writes and their constants
    double rq[TILES][2], rqinv[TILES][2], rc32[TILES][2];
#pragma unroll
    for (int t = 0; t < TILES; t++)
#pragma unroll
        for (int h = 0; h < 2; h++) {
            const uint32_t i = 16 * t + g + 8 * h;
            live[t][h] = i < level;
            const uint32_t pi = live[t][h] ? i : 0;
            fp[t][h] = pcs[pi].q < FESC_FP_LIMIT;
            rq[t][h] = pcs[pi].qd, rqinv[t][h] = pcs[pi].qinvd;
            rc32[t][h] = fp_reduce(4294967296.0, rq[t][h], rqinv[t][h]);
        }
BC_UNROLL_N(BC_UNROLL)
    for (int grp = 0; grp < BC_COEFS / 8; grp++) {
        const uint32_t c = c_base + grp * 8;
        const u64 y = has ? shoup(raw[grp], inv, invs, pk) : 0;
        // how many of the coefficient's residues are taken negative: sum over the four lanes of the coefficient, then
        // fetched for the two coefficients this lane writes
        uint32_t cnt = (has && y > half) ? 1u : 0u;
        cnt += __shfl_xor_sync(0xffffffffu, cnt, 1);
        cnt += __shfl_xor_sync(0xffffffffu, cnt, 2);
        const uint32_t cnt0 = __shfl_sync(0xffffffffu, cnt, 8 * tg), cnt1 = __shfl_sync(0xffffffffu, cnt, 8 * tg + 4);
        u64 lo[TILES][4], hi[TILES][4];
        bconv_mma<TILES>(y, sfrag, lane, lo, hi, z0, z1, z2, z3);
#pragma unroll
        for (int t = 0; t < TILES; t++)
#pragma unroll
            for (int h = 0; h < 2; h++) {
                if (!live[t][h]) continue;
                const uint32_t i = 16 * t + g + 8 * h;
                u64 w0, w1;
                if (fp[t][h]) {
                    const double q = rq[t][h], qinv = rqinv[t][h], c32 = rc32[t][h];
                    const double s0 = bconv_fp(lo[t][2 * h], hi[t][2 * h], c32, q, qinv) - tab->wrapd[cnt0][i];
                    const double s1 = bconv_fp(lo[t][2 * h + 1], hi[t][2 * h + 1], c32, q, qinv) - tab->wrapd[cnt1][i];
                    w0 = out_double ? fp_handoff(s0, q, qinv) : fp_store(s0, q, qinv);
                    w1 = out_double ? fp_handoff(s1, q, qinv) : fp_store(s1, q, qinv);
                } else {
                    const PrimeConst pc = pcs[i];
                    w0 = submod(bconv_int(lo[t][2 * h], hi[t][2 * h], pc), tab->wrap[cnt0][i], pc.q);
                    w1 = submod(bconv_int(lo[t][2 * h + 1], hi[t][2 * h + 1], pc), tab->wrap[cnt1][i], pc.q);
                }
                *reinterpret_cast<ulonglong2*>(out + (size_t)i * N + c) = make_ulonglong2(w0, w1);
            }
    }
}

bool bconv_supported(const fesc_ctx* ctx, uint32_t level) {
    static const bool on = !(getenv("FESC_BCONV") && atoi(getenv("FESC_BCONV")) == 0);   // 0: the scalar kernels (experiments)
    return on && ctx->tabs.d_md_frag && ctx->N % (BC_WARPS * BC_COEFS) == 0 && ctx->n_p <= 4 && level <= 32;
}

void moddown_conv_imma_launch(fesc_ctx* ctx, const u64* acc, u64* u, uint32_t level, uint32_t batch, int out_double, cudaStream_t st) {
    const uint32_t N = ctx->N, K = ctx->n_p;
    dim3 grid(N / (BC_WARPS * BC_COEFS), batch * 2);
    if (level > 16)
        k_moddown_conv_imma<2><<<grid, 32 * BC_WARPS, 0, st>>>(acc, u, ctx->tabs.d_moddown, ctx->tabs.d_md_frag, ctx->d_pc, N, level, ctx->n_q, K, out_double);
    else
        k_moddown_conv_imma<1><<<grid, 32 * BC_WARPS, 0, st>>>(acc, u, ctx->tabs.d_moddown, ctx->tabs.d_md_frag, ctx->d_pc, N, level, ctx->n_q, K, out_double);
}
