// Ciphertext operations: ct-pt MAC, Galois automorphism, hybrid key switch, rotation,
// rescale, ct x ct.  Every kernel streams limb rows of N words with coalesced accesses;
// products of two data words are accumulated lazily in 128 bits and reduced once.
#define FESC_DBG_FILE 3   // file id in the sites a debug build reports
#include "ops.cuh"

// ---------------------------------------------------------------------------------------
// ct-pt multiply-accumulate:  acc[b][p][l][c] += ct[b][p][l][c] * pt[b][l][c]
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_ct_pt_mac(const u64* __restrict__ ct, const u64* __restrict__ pt, size_t pt_stride,
                                                   u64* __restrict__ acc, const PrimeConst* __restrict__ pcs,
                                                   uint32_t N, uint32_t n_limbs) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t l = blockIdx.y, b = blockIdx.z;
    if (c >= N) return;
    const PrimeConst pc = pcs[l];
    const size_t poly = (size_t)n_limbs * N;
    const size_t o = (size_t)b * 2 * poly + (size_t)l * N + c;
    if (!DBG_REGION(pt + (size_t)b * pt_stride + (size_t)l * N, N * sizeof(u64))) return;
    for (int p = 0; p < 2; p++)
        if (!DBG_REGION(ct + o - c + p * poly, N * sizeof(u64)) || !DBG_REGION(acc + o - c + p * poly, N * sizeof(u64))) return;
    const u64 w = pt[(size_t)b * pt_stride + (size_t)l * N + c];
#pragma unroll
    for (int p = 0; p < 2; p++) {
        acc128 a{acc[o + p * poly], 0};
        mac128(a, ct[o + p * poly], w);
        acc[o + p * poly] = reduce128(a.hi, a.lo, pc);
    }
}

extern "C" int fesc_ct_pt_mac(fesc_ctx* ctx, const uint64_t* d_ct, const uint64_t* d_pt, size_t pt_stride,
                              uint64_t* d_acc, uint32_t batch, uint32_t n_limbs, void* stream) {
    if (!ctx || !d_ct || !d_pt || !d_acc) return FESC_EINVAL;
    if (n_limbs == 0 || n_limbs > ctx->n_q) return fesc_fail(ctx, FESC_ELEVEL, "ct_pt_mac: level out of range");
    if (batch == 0) return FESC_OK;
    if (batch > 65535) return fesc_fail(ctx, FESC_EINVAL, "ct_pt_mac: batch too large");
    dim3 grid((ctx->N + 255) / 256, n_limbs, batch);
    prof_begin(ctx, PF_POINTWISE, (cudaStream_t)stream);
    k_ct_pt_mac<<<grid, 256, 0, (cudaStream_t)stream>>>((const u64*)d_ct, (const u64*)d_pt, pt_stride, (u64*)d_acc,
                                                        ctx->d_pc, ctx->N, n_limbs);
    prof_end(ctx, PF_POINTWISE, (cudaStream_t)stream);
    FESC_CHECK_CUDA(ctx, cudaGetLastError());
    ctx->counters[2] += batch;
    return FESC_OK;
}

// ---------------------------------------------------------------------------------------
// NTT entry points
// ---------------------------------------------------------------------------------------
static int ntt_api(fesc_ctx* ctx, uint64_t* d_data, uint32_t batch, uint32_t first_limb, uint32_t n_limbs,
                   void* stream, bool inv) {
    if (!ctx || !d_data) return FESC_EINVAL;
    if (n_limbs == 0 || first_limb + n_limbs > ctx->n_primes || n_limbs > sizeof(RowMap::prime))
        return fesc_fail(ctx, FESC_EINVAL, "ntt: limb range out of bounds");
    RowMap map;
    map.period = n_limbs;
    for (uint32_t i = 0; i < n_limbs; i++) map.prime[i] = (uint8_t)(first_limb + i);
    return ntt_launch(ctx, (u64*)d_data, (size_t)batch * n_limbs, map, inv, (cudaStream_t)stream);
}
extern "C" int fesc_ntt(fesc_ctx* ctx, uint64_t* d_data, uint32_t batch, uint32_t first_limb, uint32_t n_limbs,
                        void* stream) {
    return ntt_api(ctx, d_data, batch, first_limb, n_limbs, stream, false);
}
extern "C" int fesc_intt(fesc_ctx* ctx, uint64_t* d_data, uint32_t batch, uint32_t first_limb, uint32_t n_limbs,
                         void* stream) {
    return ntt_api(ctx, d_data, batch, first_limb, n_limbs, stream, true);
}

// ---------------------------------------------------------------------------------------
// Galois automorphism in evaluation order: out[t] = in[pi_g(t)],
// pi_g(t) = brev(((2 brev(t) + 1) g mod 2N - 1) / 2).  Aligned blocks map to aligned blocks,
// so a warp reading 32 consecutive t touches one 256-byte block of the source.
// c0 goes to out0 (the result's first polynomial), c1 goes to BOTH d (kept in EVAL form for
// the digit's own limbs) and dcoef (transformed in place afterwards).
// ---------------------------------------------------------------------------------------
// Where the EVAL-form polynomial being switched is kept: the rows of the extended-digit buffer that belong to a
// digit's own limbs (row l of digit l / alpha), which the basis extension leaves untouched.  The inner product then
// reads every (digit, row) from one array.
struct OwnRows {
    u64* ext;
    uint32_t alpha, beta, rows;
    int as_double;   // rows on primes below 2^50 are kept as doubles with |x| <= q/2 (the FP64 inner product's format)
};
__device__ __forceinline__ u64 own_word(const OwnRows& w, u64 v, const PrimeConst& pc) {
    return (w.as_double && pc.q < FESC_FP_LIMIT) ? (u64)__double_as_longlong(fp_load(v, pc.qd)) : v;
}
__device__ __forceinline__ size_t own_index(const OwnRows& w, uint32_t b, uint32_t l, uint32_t N) {
    return (((size_t)b * w.beta + l / w.alpha) * w.rows + l) * N;
}
struct KsScratch;
__global__ void __launch_bounds__(256) k_autom_ct(const u64* __restrict__ in, size_t in_stride, u64* __restrict__ out0,
                                                  size_t out_stride, OwnRows d, u64* __restrict__ dcoef,
                                                  uint32_t log_n, uint32_t level, u64 g,
                                                  const PrimeConst* __restrict__ pcs, int accumulate) {
    const uint32_t N = 1u << log_n;
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t l = blockIdx.y, b = blockIdx.z;
    if (t >= N) return;
    const uint32_t src = galois_src(t, log_n, g);
    const u64* ib = in + (size_t)b * in_stride;
    const size_t poly = (size_t)level * N;
    if (src >= N || !DBG_REGION(ib + poly + (size_t)l * N, N * sizeof(u64)) ||
        !DBG_REGION(d.ext + own_index(d, b, l, N), N * sizeof(u64)) || !DBG_REGION(dcoef + ((size_t)b * level + l) * N, N * sizeof(u64)))
        return;
    const u64 v = ib[poly + (size_t)l * N + src];       // requested before the c0 part so that both gathers are in flight together
    if (out0) {        // nullptr: sigma_g(c0) is added later by the division's epilogue
        u64* o0 = out0 + (size_t)b * out_stride + (size_t)l * N + t;
        if (!DBG_REGION(ib + (size_t)l * N, N * sizeof(u64)) || !DBG_REGION(o0 - t, N * sizeof(u64))) return;
        u64 v0 = ib[(size_t)l * N + src];
        if (accumulate) v0 = addmod(v0, *o0, pcs[l].q);
        *o0 = v0;
    }
    d.ext[own_index(d, b, l, N) + t] = own_word(d, v, pcs[l]);
    dcoef[((size_t)b * level + l) * N + t] = v;
}

// ---------------------------------------------------------------------------------------
// ModUp: per digit j, uncorrected fast basis conversion of the digit's COEFF residues to every
// other active modulus and to the special moduli.
//   y_a = d_a * (Q_j/q_a)^-1 mod q_a   (canonical)
//   ext[b][j][t] = sum_a y_a * ((Q_j/q_a) mod q_t) mod q_t
// ext row order: data limbs 0..level-1 then the K special limbs; rows of the digit's own limbs
// are left untouched (the inner product reads those from the EVAL-form input).
// ---------------------------------------------------------------------------------------
// VEC (1, 2 or 4) adjacent words with 16-byte accesses where possible
template <int VEC>
__device__ __forceinline__ void ldv(const u64* __restrict__ src, u64 (&w)[VEC]) {
    if (VEC == 1) {
        w[0] = *src;
    } else {
#pragma unroll
        for (int v = 0; v < VEC / 2; v++) {
            const ulonglong2 t2 = reinterpret_cast<const ulonglong2*>(src)[v];
            w[2 * v] = t2.x, w[(2 * v + 1) % VEC] = t2.y;
        }
    }
}
template <int VEC>
__device__ __forceinline__ void stv(u64* __restrict__ dst, const u64 (&r)[VEC]) {
    if (VEC == 1) {
        *dst = r[0];
    } else {
#pragma unroll
        for (int v = 0; v < VEC / 2; v++) reinterpret_cast<ulonglong2*>(dst)[v] = make_ulonglong2(r[2 * v], r[(2 * v + 1) % VEC]);
    }
}

template <int ALPHA, int VEC>
__global__ void __launch_bounds__(256) k_modup(const u64* __restrict__ dcoef, u64* __restrict__ ext,
                                               const ModUpDigit* __restrict__ tab, const PrimeConst* __restrict__ pcs,
                                               uint32_t N, uint32_t level, uint32_t n_q, uint32_t K, uint32_t beta,
                                               int out_double) {
    // VEC adjacent coefficients per thread: every table word and every prime constant serves VEC products
    const uint32_t c = (blockIdx.x * blockDim.x + threadIdx.x) * VEC;
    const uint32_t j = blockIdx.y, b = blockIdx.z;
    if (c >= N) return;
    const ModUpDigit* dg = tab + j;
    const uint32_t first = dg->first, n_src = dg->n_src;
    if (!DBG_REGION(dg, sizeof(ModUpDigit)) || !DBG_REGION(dcoef + ((size_t)b * level + first) * N, (size_t)n_src * N * sizeof(u64)) ||
        !DBG_REGION(ext + ((size_t)b * beta + j) * (level + K) * N, (size_t)(level + K) * N * sizeof(u64)))
        return;
    u64 y[ALPHA][VEC];
    bool src_small = true;
#pragma unroll
    for (int a = 0; a < ALPHA; a++) {
#pragma unroll
        for (int v = 0; v < VEC; v++) y[a][v] = 0;
        if (a < n_src) {
            const u64* src = dcoef + ((size_t)b * level + first + a) * N + c;
            const u64 q = pcs[first + a].q, inv = dg->inv[a], invs = dg->invs[a];
            src_small = src_small && q < FESC_FP_LIMIT;
            u64 w[VEC];
            ldv<VEC>(src, w);
#pragma unroll
            for (int v = 0; v < VEC; v++) y[a][v] = shoup(w[v], inv, invs, q);
        }
    }
    const uint32_t rows = level + K;
    u64* out = ext + ((size_t)b * beta + j) * rows * N + c;
    // every y_a is below 2^50 when its source prime is: exact FP64 products for targets below 2^50
    double yd[ALPHA][VEC];
#pragma unroll
    for (int a = 0; a < ALPHA; a++)
#pragma unroll
        for (int v = 0; v < VEC; v++) yd[a][v] = fp_from_u64(y[a][v] & 0x000FFFFFFFFFFFFFull);
    for (uint32_t t = 0; t < rows; t++) {
        if (t >= first && t < first + n_src) continue;
        const uint32_t pt = t < level ? t : n_q + (t - level);
        u64 r[VEC];
        if (src_small && pcs[pt].q < FESC_FP_LIMIT) {
            const double q = pcs[pt].qd, qinv = pcs[pt].qinvd;
            double s[VEC];
#pragma unroll
            for (int v = 0; v < VEC; v++) s[v] = 0.0;
#pragma unroll
            for (int a = 0; a < ALPHA; a++)
                if (a < n_src) {
                    const double m = dg->matd[a][pt];
#pragma unroll
                    for (int v = 0; v < VEC; v++) s[v] += fp_modmul(yd[a][v], m, q, qinv);
                }
#pragma unroll
            for (int v = 0; v < VEC; v++) r[v] = out_double ? fp_handoff(s[v], q, qinv) : fp_store(s[v], q, qinv);
        } else {
            const PrimeConst pc = pcs[pt];
#pragma unroll
            for (int v = 0; v < VEC; v++) {
                acc128 acc{0, 0};
#pragma unroll
                for (int a = 0; a < ALPHA; a++)
                    if (a < n_src) mac128(acc, y[a][v], dg->mat[a][pt]);
                r[v] = reduce128(acc.hi, acc.lo, pc);
                // the hand-over format follows the TARGET prime (the transform picks its arithmetic by that prime)
                if (out_double && pc.q < FESC_FP_LIMIT) r[v] = (u64)__double_as_longlong(fp_load(r[v], pc.qd));
            }
        }
        stv<VEC>(out + (size_t)t * N, r);
    }
}

// ---------------------------------------------------------------------------------------
// Inner product with the switching key over all level+K moduli:
//   acc[b][p][t] = sum_j dt_j[b][t] * key[j][p][t],   dt_j[t] = d[b][t] if t is in digit j, else ext[b][j][t].
// One thread owns one (coefficient, modulus) and BT ciphertexts, so a key word is loaded once
// for BT products.
// ---------------------------------------------------------------------------------------
// coefficients per thread of the basis-conversion kernels
#ifndef KS_VEC
#define KS_VEC 2
#endif
#ifndef INNER_MINB
#define INNER_MINB 4
#endif
// Several sources can be summed in one pass: source s contributes sum_j dt_j(ext_s)[pi_{g_s}(t)] * key_s[j].  The giant
// steps of a projection (different converted polynomials, different keys, one sum) and the rotate-and-add chains (one
// converted polynomial read through several Galois permutations, one key each) then read and write the accumulators
// once instead of once per key, and the later reads of a shared source hit L2.
#define INNER_MAX_SRC 8
struct InnerSrc {
    const u64* ext;   // [batch][beta][level+K][N]
    const u64* key;   // [beta][2][n_q+K][N]
    u64 g;            // Galois element the digits are read through (0: none)
};
struct InnerSrcs {
    InnerSrc s[INNER_MAX_SRC];
    uint32_t n;
};
// PATH 0: the row's prime decides at run time; 1: the caller guarantees primes below 2^50 on rows
// [row0, row0 + gridDim.y) (exact FP64 products only); 2: the caller sends those rows to the 128-bit integer sums.
template <int BT, int PATH>
__global__ void __launch_bounds__(256, INNER_MINB) k_inner(InnerSrcs S, u64* __restrict__ acc,
                                               const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level,
                                               uint32_t n_q, uint32_t K, uint32_t alpha, uint32_t beta,
                                               uint32_t batch, uint32_t log_n, int accumulate, uint32_t row0,
                                               int x_double) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t t = row0 + blockIdx.y, b0 = blockIdx.z * BT;
    if (c >= N) return;
    const uint32_t rows = level + K, np = n_q + K;
    const uint32_t pt = t < level ? t : n_q + (t - level);
    // operand words of one digit: key (b, a) and the BT ciphertext words; clamped indices keep loads valid.
    // All addresses are a per-thread base plus a multiple of one stride (no per-load index products).
    const size_t kstride = (size_t)np * N, xstride = (size_t)rows * N;
#ifdef FESC_DEBUG_BOUNDS
    for (uint32_t s = 0; s < S.n; s++) {
        if (S.s[s].g && galois_src(c, log_n, S.s[s].g) >= N) return;
        for (uint32_t j = 0; j < beta; j++) {
            if (!DBG_REGION(S.s[s].key + ((size_t)(2 * j) * np + pt) * N, N * sizeof(u64)) ||
                !DBG_REGION(S.s[s].key + ((size_t)(2 * j + 1) * np + pt) * N, N * sizeof(u64)))
                return;
            for (int i = 0; i < BT; i++) {
                const uint32_t b = b0 + i < batch ? b0 + i : batch - 1;
                if (!DBG_REGION(S.s[s].ext + (((size_t)b * beta + j) * rows + t) * N, N * sizeof(u64))) return;
            }
        }
    }
    for (int i = 0; i < BT; i++) {
        const uint32_t b = b0 + i < batch ? b0 + i : batch - 1;
        if (!DBG_REGION(acc + (((size_t)b * 2 + 0) * rows + t) * N, N * sizeof(u64)) ||
            !DBG_REGION(acc + (((size_t)b * 2 + 1) * rows + t) * N, N * sizeof(u64)))
            return;
    }
#endif
    // the (source, digit) whose words are requested next; hoisted rotations: the automorphism acts on the extended
    // digits, i.e. they are read at pi_g(c)
    uint32_t sn = 0, jn = 0;
    const u64* kp;
    const u64* xp[BT];
    auto setup = [&](uint32_t s) {
        const u64 g = S.s[s].g;
        const uint32_t cs = g ? galois_src(c, log_n, g) : c;
        kp = S.s[s].key + (size_t)pt * N + c;
#pragma unroll
        for (int i = 0; i < BT; i++) {
            const uint32_t b = b0 + i < batch ? b0 + i : batch - 1;
            xp[i] = S.s[s].ext + ((size_t)b * beta * rows + t) * N + cs;
        }
    };
    auto load_next = [&](u64& kb, u64& ka, u64 (&x)[BT]) {
        kb = __ldg(kp + (size_t)(2 * jn) * kstride);
        ka = __ldg(kp + (size_t)(2 * jn + 1) * kstride);
#pragma unroll
        for (int i = 0; i < BT; i++) x[i] = xp[i][(size_t)jn * xstride];
        if (++jn == beta) {
            jn = 0;
            if (++sn < S.n) setup(sn);
        }
    };
    const uint32_t total = S.n * beta;
    setup(0);
    if (PATH == 1 || (PATH == 0 && pcs[pt].q < FESC_FP_LIMIT)) {
        // exact FP64 products of canonical words (both below q): every product is below 0.875q, so a running sum of
        // at most q/2 plus 7 terms stays below 2^53 = 8q; longer sums are folded back after every 7th term.  The next digit's words
        // are requested before this digit's products start: 2 + BT loads in flight per thread, few registers,
        // so that four CTAs per SM overlap their loads and products (measured: one digit ahead with 4 CTAs of 4
        // ciphertexts per thread moves 1.6x the bytes per second of all-digits-up-front with 2 CTAs; 8 ciphertexts
        // per thread with 2 CTAs and 2 per thread with 6 CTAs are both slower).
        const double q = pcs[pt].qd, qinv = pcs[pt].qinvd;
        double f0[BT], f1[BT];
#pragma unroll
        for (int i = 0; i < BT; i++) {
            f0[i] = f1[i] = 0.0;
            if (accumulate) {   // running sum over several passes (division by P deferred)
                const uint32_t b = b0 + i < batch ? b0 + i : batch - 1;
                f0[i] = fp_load(acc[(((size_t)b * 2 + 0) * rows + t) * N + c], q);
                f1[i] = fp_load(acc[(((size_t)b * 2 + 1) * rows + t) * N + c], q);
            }
        }
        u64 kb, ka, x[BT], nkb = 0, nka = 0, nx[BT];
#pragma unroll
        for (int i = 0; i < BT; i++) nx[i] = 0;
        load_next(kb, ka, x);
#pragma unroll 1
        for (uint32_t it = 0; it < total; it++) {
            if (it + 1 < total) load_next(nkb, nka, nx);
            const double dkb = fp_from_u64(kb), dka = fp_from_u64(ka);
#pragma unroll
            for (int i = 0; i < BT; i++) {
                // canonical words (every product below 0.875q) or doubles with |x| <= q/2 left by the producers
                const double xd = x_double ? __longlong_as_double((long long)x[i]) : fp_from_u64(x[i]);
                f0[i] += fp_modmul(xd, dkb, q, qinv);
                f1[i] += fp_modmul(xd, dka, q, qinv);
            }
            if (it % 7 == 6) {   // |running sum| <= q/2 plus 7 products below 0.875q each stays below 6.7q < 2^53: fold after every 7th
#pragma unroll
                for (int i = 0; i < BT; i++) {
                    f0[i] = fp_reduce(f0[i], q, qinv);
                    f1[i] = fp_reduce(f1[i], q, qinv);
                }
            }
            kb = nkb, ka = nka;
#pragma unroll
            for (int i = 0; i < BT; i++) x[i] = nx[i];
        }
#pragma unroll
        for (int i = 0; i < BT; i++) {
            const uint32_t b = b0 + i;
            if (b < batch) {
                acc[(((size_t)b * 2 + 0) * rows + t) * N + c] = fp_store(f0[i], q, qinv);
                acc[(((size_t)b * 2 + 1) * rows + t) * N + c] = fp_store(f1[i], q, qinv);
            }
        }
        return;
    }
    if (PATH != 1) {
        const PrimeConst pc = pcs[pt];
        acc128 a0[BT], a1[BT];
#pragma unroll
        for (int i = 0; i < BT; i++) a0[i] = a1[i] = acc128{0, 0};
        {
            u64 kb, ka, x[BT], nkb = 0, nka = 0, nx[BT];
#pragma unroll
            for (int i = 0; i < BT; i++) nx[i] = 0;
            load_next(kb, ka, x);
#pragma unroll 1
            for (uint32_t it = 0; it < total; it++) {
                if (it + 1 < total) load_next(nkb, nka, nx);
#pragma unroll
                for (int i = 0; i < BT; i++) {
                    mac128(a0[i], x[i], kb);
                    mac128(a1[i], x[i], ka);
                }
                if ((it & 7) == 7 && it + 1 < total) {   // 8 products below 2^124 cannot wrap 128 bits: longer sums are reduced in between
#pragma unroll
                    for (int i = 0; i < BT; i++) {
                        a0[i] = acc128{reduce128(a0[i].hi, a0[i].lo, pc), 0};
                        a1[i] = acc128{reduce128(a1[i].hi, a1[i].lo, pc), 0};
                    }
                }
                kb = nkb, ka = nka;
#pragma unroll
                for (int i = 0; i < BT; i++) x[i] = nx[i];
            }
        }
#pragma unroll
        for (int i = 0; i < BT; i++) {
            const uint32_t b = b0 + i;
            if (b < batch) {
                u64* o0 = acc + (((size_t)b * 2 + 0) * rows + t) * N + c;
                u64* o1 = acc + (((size_t)b * 2 + 1) * rows + t) * N + c;
                u64 r0 = reduce128(a0[i].hi, a0[i].lo, pc), r1 = reduce128(a1[i].hi, a1[i].lo, pc);
                if (accumulate) r0 = addmod(r0, *o0, pc.q), r1 = addmod(r1, *o1, pc.q);
                *o0 = r0;
                *o1 = r1;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------
// The same inner product with operands staged by bulk asynchronous copies (TMA; every copy targets this CTA only).
// A persistent CTA walks over tiles (limb row t, 256 coefficients, BT ciphertexts).  One thread requests, per
// digit, the two key rows and the BT digit rows of the NEXT tile (2 KB each) into the other half of shared memory,
// completion counted in bytes on an mbarrier, while all threads multiply out the current tile from shared memory;
// nothing is staged through registers, so one CTA keeps 2 x beta x (2 + BT) x 2 KB in flight.  Tiles that share key
// rows (same row and coefficient block, other ciphertext group) are adjacent in the tile order, i.e. run at the
// same time on neighbouring SMs and share the key through L2.  For hoisted rotations the source block of the
// digit rows is the image of the coefficient block under the Galois permutation (aligned blocks map to aligned
// blocks) and a thread picks its word inside the block.  Every wait is bounded: a wait that runs out sets the
// status word and the CTA returns.
// ---------------------------------------------------------------------------------------
// Self-test of the bounded wait: one warp waits on a barrier phase that nothing completes, with a small poll budget;
// the wait runs out, the status word is set and the kernel returns (no copy is in flight, nothing faults).
__global__ void k_wait_limit_selftest(uint32_t* __restrict__ status) {
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t b = (uint32_t)__cvta_generic_to_shared(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    uint32_t late = 1;
    for (uint32_t it = 0; it < 4096 && late; it++) {
        late = !mbar_try_wait(b, 0);
        if (late) __nanosleep(32);
    }
    if (__any_sync(0xffffffffu, late) && threadIdx.x == 0) atomicExch(status, 2u);
}
extern "C" int fesc_selftest_wait_limit(fesc_ctx* ctx, void* stream) {
    if (!ctx) return FESC_EINVAL;
    k_wait_limit_selftest<<<1, 32, 0, (cudaStream_t)stream>>>(ctx->d_status);
    FESC_CHECK_CUDA(ctx, cudaGetLastError());
    return FESC_OK;
}

template <int BT>
__global__ void __launch_bounds__(256, 1) k_inner_tma(const u64* __restrict__ ext,
                                                      const u64* __restrict__ key, u64* __restrict__ acc,
                                                      const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level,
                                                      uint32_t n_q, uint32_t K, uint32_t alpha, uint32_t beta,
                                                      uint32_t batch, uint32_t log_n, u64 g, int accumulate,
                                                      uint32_t n_tiles, uint32_t* __restrict__ status, int x_double) {
    constexpr int R = 2 + BT;                                // rows per digit: key b, key a, BT ciphertexts
    extern __shared__ __align__(128) u64 smem[];             // [2 stages][beta][R][256] then two barriers
    const uint32_t tid = threadIdx.x;
    const uint32_t rows = level + K, np = n_q + K, nblk = N >> 8, ngrp = (batch + BT - 1) / BT;
    const uint32_t stage_words = beta * R * 256;
    const uint32_t sbase = (uint32_t)__cvta_generic_to_shared(smem);
    const uint32_t bar0 = sbase + 2 * stage_words * 8;
    if (tid == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    auto decode = [&](uint32_t tile, uint32_t& t, uint32_t& cblk, uint32_t& b0) {
        const uint32_t grp = tile % ngrp, rest = tile / ngrp;
        cblk = rest % nblk;
        t = rest / nblk;
        b0 = grp * BT;
    };
    auto issue = [&](uint32_t tile, uint32_t stage) {        // thread 0 only
        uint32_t t, cblk, b0;
        decode(tile, t, cblk, b0);
        const uint32_t pt = t < level ? t : n_q + (t - level);
        const uint32_t sblk = g ? (galois_src(cblk << 8, log_n, g) >> 8) : cblk;
        const uint32_t bar = bar0 + stage * 8;
        uint32_t dst = sbase + stage * stage_words * 8;
#ifdef FESC_DEBUG_BOUNDS
        for (uint32_t j = 0; j < beta; j++) {      // a bad source: no copy is issued, the wait below runs out and the CTA returns
            if (!DBG_REGION(key + ((size_t)(2 * j) * np + pt) * N + (cblk << 8), 2048) ||
                !DBG_REGION(key + ((size_t)(2 * j + 1) * np + pt) * N + (cblk << 8), 2048))
                return;
            for (int i = 0; i < BT; i++) {
                const uint32_t b = b0 + i < batch ? b0 + i : batch - 1;
                if (!DBG_REGION(ext + (((size_t)b * beta + j) * rows + t) * N + (sblk << 8), 2048)) return;
            }
        }
#endif
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier reads of this half precede the refill
        mbar_expect_tx(bar, stage_words * 8);
        for (uint32_t j = 0; j < beta; j++) {
            bulk_g2s(dst, key + ((size_t)(2 * j) * np + pt) * N + (cblk << 8), 2048, bar);
            bulk_g2s(dst + 2048, key + ((size_t)(2 * j + 1) * np + pt) * N + (cblk << 8), 2048, bar);
            dst += 4096;
#pragma unroll
            for (int i = 0; i < BT; i++) {
                const uint32_t b = b0 + i < batch ? b0 + i : batch - 1;
                const u64* src = ext + (((size_t)b * beta + j) * rows + t) * N;
                bulk_g2s(dst, src + (sblk << 8), 2048, bar);
                dst += 2048;
            }
        }
    };
    uint32_t tile = blockIdx.x;
    if (tid == 0 && tile < n_tiles) issue(tile, 0);
    for (uint32_t k = 0; tile < n_tiles; k++, tile += gridDim.x) {
        const uint32_t stage = k & 1;
        if (tid == 0 && tile + gridDim.x < n_tiles) issue(tile + gridDim.x, stage ^ 1);
        const uint32_t late = mbar_wait_bounded(bar0 + stage * 8, (k >> 1) & 1);
        if (__syncthreads_or((int)late)) {                   // block-uniform: give up together
            if (tid == 0) {
                atomicExch(status, 1u);
                // copies may still be in flight into this CTA's shared memory: one more bounded wait on the stage
                // that ran out and one on the other stage before the memory can be handed to another CTA (after a
                // time-out the caller has to synchronise and discard whatever overlapped on the device anyway)
                mbar_wait_bounded(bar0 + stage * 8, (k >> 1) & 1);
                if (tile + gridDim.x < n_tiles) mbar_wait_bounded(bar0 + (stage ^ 1) * 8, ((k + 1) >> 1) & 1);
            }
            return;
        }
        uint32_t t, cblk, b0;
        decode(tile, t, cblk, b0);
        const uint32_t c = (cblk << 8) + tid;
#ifdef FESC_DEBUG_BOUNDS
        {
            bool ok = true;                                  // the same for every thread of the CTA
            for (int i = 0; i < BT; i++) {
                const uint32_t b = b0 + i < batch ? b0 + i : batch - 1;
                ok = ok && DBG_REGION(acc + (((size_t)b * 2 + 0) * rows + t) * N + (cblk << 8), 2048) &&
                     DBG_REGION(acc + (((size_t)b * 2 + 1) * rows + t) * N + (cblk << 8), 2048);
            }
            if (!ok) {
                __syncthreads();
                continue;
            }
        }
#endif
        const uint32_t si = g ? (galois_src(c, log_n, g) & 255u) : tid;
        const uint32_t pt = t < level ? t : n_q + (t - level);
        const u64* sm = smem + (size_t)stage * stage_words;
        if (pcs[pt].q < FESC_FP_LIMIT) {
            const double q = pcs[pt].qd, qinv = pcs[pt].qinvd;
            double f0[BT], f1[BT];
#pragma unroll
            for (int i = 0; i < BT; i++) {
                f0[i] = f1[i] = 0.0;
                if (accumulate) {
                    const uint32_t b = b0 + i < batch ? b0 + i : batch - 1;
                    f0[i] = fp_load(acc[(((size_t)b * 2 + 0) * rows + t) * N + c], q);
                    f1[i] = fp_load(acc[(((size_t)b * 2 + 1) * rows + t) * N + c], q);
                }
            }
            for (uint32_t j = 0; j < beta; j++) {
                const u64* dj = sm + (size_t)j * R * 256;
                const double dkb = fp_from_u64(dj[tid]), dka = fp_from_u64(dj[256 + tid]);
#pragma unroll
                for (int i = 0; i < BT; i++) {
                    const u64 xw = dj[(2 + i) * 256 + si];
                    const double xd = x_double ? __longlong_as_double((long long)xw) : fp_load(xw, q);
                    f0[i] += fp_modmul(xd, dkb, q, qinv);
                    f1[i] += fp_modmul(xd, dka, q, qinv);
                }
                if (j % 7 == 6) {   // same schedule as k_inner: |sum| <= q/2 plus 7 products stays below 6.7q
#pragma unroll
                    for (int i = 0; i < BT; i++) {
                        f0[i] = fp_reduce(f0[i], q, qinv);
                        f1[i] = fp_reduce(f1[i], q, qinv);
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < BT; i++) {
                const uint32_t b = b0 + i;
                if (b < batch) {
                    acc[(((size_t)b * 2 + 0) * rows + t) * N + c] = fp_store(f0[i], q, qinv);
                    acc[(((size_t)b * 2 + 1) * rows + t) * N + c] = fp_store(f1[i], q, qinv);
                }
            }
        } else {
            const PrimeConst pc = pcs[pt];
            acc128 a0[BT], a1[BT];
#pragma unroll
            for (int i = 0; i < BT; i++) a0[i] = a1[i] = acc128{0, 0};
            for (uint32_t j = 0; j < beta; j++) {
                const u64* dj = sm + (size_t)j * R * 256;
                const u64 kb = dj[tid], ka = dj[256 + tid];
#pragma unroll
                for (int i = 0; i < BT; i++) {
                    const u64 x = dj[(2 + i) * 256 + si];
                    mac128(a0[i], x, kb);
                    mac128(a1[i], x, ka);
                }
            }
#pragma unroll
            for (int i = 0; i < BT; i++) {
                const uint32_t b = b0 + i;
                if (b < batch) {
                    u64* o0 = acc + (((size_t)b * 2 + 0) * rows + t) * N + c;
                    u64* o1 = acc + (((size_t)b * 2 + 1) * rows + t) * N + c;
                    u64 r0 = reduce128(a0[i].hi, a0[i].lo, pc), r1 = reduce128(a1[i].hi, a1[i].lo, pc);
                    if (accumulate) r0 = addmod(r0, *o0, pc.q), r1 = addmod(r1, *o1, pc.q);
                    *o0 = r0;
                    *o1 = r1;
                }
            }
        }
        __syncthreads();                                     // this half may be refilled from now on
    }
}

// ---------------------------------------------------------------------------------------
// Division by P, conversion step: special-limb residues (COEFF) -> u[b][p][i] (COEFF, data limbs)
//   y_k = r_k * (P/p_k)^-1 mod p_k, taken in [-(p_k-1)/2, (p_k-1)/2];
//   u_i = sum_k y_k (P/p_k) mod q_i = sum_k [y_k]_canonical (P/p_k) - #{y_k > p_k/2} * P  (mod q_i).
// ---------------------------------------------------------------------------------------
template <int VEC>
__global__ void __launch_bounds__(256) k_moddown_conv(const u64* __restrict__ acc, u64* __restrict__ u,
                                                      const ModDownTab* __restrict__ tab,
                                                      const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level,
                                                      uint32_t n_q, uint32_t K, int out_double) {
    // VEC adjacent coefficients per thread: every table word and every prime constant serves VEC products
    const uint32_t c = (blockIdx.x * blockDim.x + threadIdx.x) * VEC;
    const uint32_t bp = blockIdx.y;   // b*2 + p
    if (c >= N) return;
    const uint32_t rows = level + K;
    if (!DBG_REGION(acc + ((size_t)bp * rows + level) * N, (size_t)K * N * sizeof(u64)) ||
        !DBG_REGION(u + (size_t)bp * level * N, (size_t)level * N * sizeof(u64)) || !DBG_REGION(tab, sizeof(ModDownTab)))
        return;
    u64 y[FESC_MAX_SPECIAL][VEC];
    uint32_t cnt[VEC];
#pragma unroll
    for (int v = 0; v < VEC; v++) cnt[v] = 0;
#pragma unroll
    for (int k = 0; k < FESC_MAX_SPECIAL; k++) {
#pragma unroll
        for (int v = 0; v < VEC; v++) y[k][v] = 0;
        if (k < K) {
            const u64* src = acc + ((size_t)bp * rows + level + k) * N + c;
            u64 w[VEC];
            ldv<VEC>(src, w);
            const u64 inv = tab->inv[k], invs = tab->invs[k], pk = pcs[n_q + k].q, half = tab->half[k];
#pragma unroll
            for (int v = 0; v < VEC; v++) {
                y[k][v] = shoup(w[v], inv, invs, pk);
                cnt[v] += y[k][v] > half;
            }
        }
    }
    // 30-bit halves of every y_k as doubles, for targets below 2^50 (exact FP64 products)
    double yh[FESC_MAX_SPECIAL][VEC], yl[FESC_MAX_SPECIAL][VEC];
#pragma unroll
    for (int k = 0; k < FESC_MAX_SPECIAL; k++)
#pragma unroll
        for (int v = 0; v < VEC; v++) {
            yh[k][v] = fp_from_u64(y[k][v] >> 30);
            yl[k][v] = fp_from_u64(y[k][v] & ((1ull << 30) - 1));
        }
    for (uint32_t i = 0; i < level; i++) {
        u64 r[VEC];
        if (pcs[i].q < FESC_FP_LIMIT) {
            const double q = pcs[i].qd, qinv = pcs[i].qinvd;
            double s[VEC];
#pragma unroll
            for (int v = 0; v < VEC; v++) s[v] = -tab->wrapd[cnt[v]][i];
#pragma unroll
            for (int k = 0; k < FESC_MAX_SPECIAL; k++)
                if (k < K) {
                    const double m30 = tab->mat30d[k][i], m = tab->matd[k][i];
#pragma unroll
                    for (int v = 0; v < VEC; v++) {
                        s[v] += fp_modmul(yh[k][v], m30, q, qinv);
                        s[v] += fp_modmul(yl[k][v], m, q, qinv);
                        if (k == 3) s[v] = fp_reduce(s[v], q, qinv);
                    }
                }
#pragma unroll
            for (int v = 0; v < VEC; v++) r[v] = out_double ? fp_handoff(s[v], q, qinv) : fp_store(s[v], q, qinv);
        } else {
            const PrimeConst pc = pcs[i];
#pragma unroll
            for (int v = 0; v < VEC; v++) {
                acc128 a{0, 0};
#pragma unroll
                for (int k = 0; k < FESC_MAX_SPECIAL; k++)
                    if (k < K) mac128(a, y[k][v], tab->mat[k][i]);
                r[v] = submod(reduce128(a.hi, a.lo, pc), tab->wrap[cnt[v]][i], pc.q);
            }
        }
        stv<VEC>(u + ((size_t)bp * level + i) * N + c, r);
    }
}

// out[b][p][i] = (acc[b][p][i] - u[b][p][i]) * P^-1 + add[b][p][i]   (all EVAL)
__global__ void __launch_bounds__(256) k_moddown_finish(const u64* __restrict__ acc, const u64* __restrict__ u,
                                                        u64* __restrict__ out, size_t out_stride,
                                                        const ModDownTab* __restrict__ tab,
                                                        const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level,
                                                        uint32_t K, int add_mask) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t i = blockIdx.y, bp = blockIdx.z;
    if (c >= N) return;
    const uint32_t b = bp >> 1, p = bp & 1;
    const u64 q = pcs[i].q;
    u64* o = out + (size_t)b * out_stride + ((size_t)p * level + i) * N + c;
    if (!DBG_REGION(o - c, N * sizeof(u64)) || !DBG_REGION(acc + ((size_t)bp * (level + K) + i) * N, N * sizeof(u64)) ||
        !DBG_REGION(u + ((size_t)bp * level + i) * N, N * sizeof(u64)))
        return;
    const u64 av = acc[((size_t)bp * (level + K) + i) * N + c], uv = u[((size_t)bp * level + i) * N + c];
    if (q < FESC_FP_LIMIT) {
        const double qd = pcs[i].qd, qinv = pcs[i].qinvd;
        double s = fp_modmul(fp_load(av, qd) - fp_load(uv, qd), fp_from_u64(tab->pinv[i]), qd, qinv);
        if ((add_mask >> p) & 1) s += fp_load(*o, qd);
        *o = fp_store(s, qd, qinv);
        return;
    }
    u64 v = submod(av, uv, q);
    v = shoup(v, tab->pinv[i], tab->pinvs[i], q);
    if ((add_mask >> p) & 1) v = addmod(v, *o, q);
    *o = v;
}

// Steps 1-3 of the key switch: ws.dcoef -> COEFF, digit-wise basis extension into ws.ext, NTT of the
// converted rows.  The result (ws.ext, own-limb rows included) can serve several keys (hoisted rotations).
static int ks_decompose(fesc_ctx* ctx, const KsScratch& ws, uint32_t level, uint32_t batch, cudaStream_t st) {
    const uint32_t N = ctx->N, K = ctx->n_p, nq = ctx->n_q, alpha = ctx->alpha;
    const uint32_t beta = (level + alpha - 1) / alpha, rows = level + K;
    const uint32_t gx = (N + 255) / 256;
    int rc;
    RowMap m;
    // 1. d -> COEFF
    m.period = level;
    for (uint32_t i = 0; i < level; i++) m.prime[i] = (uint8_t)i;
    if ((rc = ntt_launch(ctx, ws.dcoef, (size_t)batch * level, m, true, st)) != FESC_OK) return rc;
    // 2. ModUp
    const ModUpDigit* tab = ctx->tabs.d_modup + (size_t)(level - 1) * ctx->beta_max;
    const int dbl = ctx->log_n == 16;   // the N = 2^16 forward transform takes doubles straight from the conversion
    const bool vec2 = N % (256 * KS_VEC) == 0;
    dim3 gmu(vec2 ? N / (256 * KS_VEC) : gx, beta, batch);
#define MODUP(A)                                                                                           \
    do {                                                                                                   \
        if (vec2) k_modup<A, KS_VEC><<<gmu, 256, 0, st>>>(ws.dcoef, ws.ext, tab, ctx->d_pc, N, level, nq, K, beta, dbl); \
        else k_modup<A, 1><<<gmu, 256, 0, st>>>(ws.dcoef, ws.ext, tab, ctx->d_pc, N, level, nq, K, beta, dbl);  \
    } while (0)
    prof_begin(ctx, PF_MODUP, st);
    if (alpha <= 1) MODUP(1);
    else if (alpha <= 2) MODUP(2);
    else if (alpha <= 4) MODUP(4);
    else if (alpha <= 6) MODUP(6);
    else MODUP(8);
#undef MODUP
    prof_end(ctx, PF_MODUP, st);
    // 3. NTT of the converted rows
    if (beta * rows > sizeof(RowMap::prime)) return fesc_fail(ctx, FESC_EINVAL, "key switch: too many digit rows");
    m.period = beta * rows;
    for (uint32_t j = 0; j < beta; j++)
        for (uint32_t t = 0; t < rows; t++) {
            bool own = t < level && t / alpha == j;
            m.prime[j * rows + t] = own ? 0xFF : (uint8_t)(t < level ? t : nq + (t - level));
        }
    if ((rc = ntt_launch(ctx, ws.ext, (size_t)batch * beta * rows, m, false, st, dbl != 0, dbl != 0)) != FESC_OK) return rc;
    FESC_CHECK_CUDA(ctx, cudaGetLastError());
    return FESC_OK;
}

// Step 4: inner products of the sources `S` (converted digits, key, Galois element each) summed into ws.acc;
// accumulate != 0 adds to what ws.acc holds (sums over several passes before one division by P).
static int ks_inner_multi(fesc_ctx* ctx, const KsScratch& ws, const InnerSrcs& S, uint32_t level, uint32_t batch,
                          cudaStream_t st, int accumulate) {
    const uint32_t N = ctx->N, K = ctx->n_p, nq = ctx->n_q, alpha = ctx->alpha;
    const uint32_t beta = (level + alpha - 1) / alpha, rows = level + K;
    const uint32_t gx = (N + 255) / 256;
    prof_begin(ctx, PF_INNER, st);
    const bool use_tma = S.n == 1 && getenv("FESC_INNER_TMA") != nullptr;   // read per call so a test can switch it
#define INNER(BT_, PATH_, ROW0_, NROWS_)                                                                        \
    do {                                                                                                        \
        dim3 gd(gx, NROWS_, (batch + BT_ - 1) / BT_);                                                           \
        k_inner<BT_, PATH_><<<gd, 256, 0, st>>>(S, ws.acc, ctx->d_pc, N, level, nq, K, alpha, beta, batch,     \
                                                ctx->log_n, accumulate, ROW0_, ctx->log_n == 16);              \
    } while (0)
    // data rows on primes below 2^50 and special rows above: one launch per kind, each compiled for its arithmetic
    bool split = true;
    for (uint32_t i = 0; i < level; i++) split = split && ctx->q[i] < FESC_FP_LIMIT;
    for (uint32_t k = 0; k < K; k++) split = split && ctx->q[nq + k] >= FESC_FP_LIMIT;
    if (use_tma && N % 256 == 0 && beta <= 8 && batch >= 3) {   // 128-bit sums of <= 8 products below 2^124 cannot wrap
        const uint32_t n_tiles = rows * (N >> 8) * ((batch + 3) / 4);
        const size_t smem = (size_t)2 * beta * 6 * 2048 + 16;
        int dev = 0, sms = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        FESC_CHECK_CUDA(ctx, cudaFuncSetAttribute(k_inner_tma<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        const uint32_t grid = n_tiles < (uint32_t)sms ? n_tiles : (uint32_t)sms;
        k_inner_tma<4><<<grid, 256, smem, st>>>(S.s[0].ext, S.s[0].key, ws.acc, ctx->d_pc, N, level, nq, K, alpha, beta,
                                                 batch, ctx->log_n, S.s[0].g, accumulate, n_tiles, ctx->d_status, ctx->log_n == 16);
    } else if (split) {
        if (batch >= 3) INNER(4, 1, 0, level);
        else if (batch == 2) INNER(2, 1, 0, level);
        else INNER(1, 1, 0, level);
        if (batch >= 3) INNER(4, 2, level, K);
        else if (batch == 2) INNER(2, 2, level, K);
        else INNER(1, 2, level, K);
    } else if (batch >= 3) INNER(4, 0, 0, rows);
    else if (batch == 2) INNER(2, 0, 0, rows);
    else INNER(1, 0, 0, rows);
#undef INNER
    prof_end(ctx, PF_INNER, st);
    FESC_CHECK_CUDA(ctx, cudaGetLastError());
    ctx->counters[1] += (uint64_t)batch * S.n;
    return FESC_OK;
}
// one source: ws.ext with `key`, digits read through the Galois permutation of g when g != 0
static int ks_inner(fesc_ctx* ctx, const KsScratch& ws, const EvalKey& key, uint32_t level, uint32_t batch,
                    cudaStream_t st, u64 g, int accumulate) {
    InnerSrcs S;
    S.n = 1;
    S.s[0] = InnerSrc{ws.ext, key.d_key, g};
    return ks_inner_multi(ctx, ws, S, level, batch, st, accumulate);
}

// Step 5: division of ws.acc by P; the result is ADDED to out[b][p] when bit p of add_mask is set, else stored.
// whether the last pass of the forward transform finishes the division (N = 2^16, every data prime below 2^50)
static bool moddown_fused(const fesc_ctx* ctx, uint32_t level) {
    bool fuse = ctx->log_n == 16;
    for (uint32_t i = 0; i < level; i++) fuse = fuse && ctx->q[i] < FESC_FP_LIMIT;
    return fuse;
}
// rot_src != nullptr (only when moddown_fused): out[b][0] also receives sigma_g(c0) of the ciphertext at
// rot_src + b * rot_stride, read through the permutation by the fused epilogue
static int ks_moddown(fesc_ctx* ctx, const KsScratch& ws, uint32_t level, uint32_t batch, u64* out, size_t out_stride,
                      int add_mask, cudaStream_t st, const u64* rot_src = nullptr, size_t rot_stride = 0, u64 rot_g = 0) {
    const uint32_t N = ctx->N, K = ctx->n_p, nq = ctx->n_q;
    const uint32_t rows = level + K;
    const uint32_t gx = (N + 255) / 256;
    int rc;
    RowMap m;
    m.period = rows;
    for (uint32_t t = 0; t < rows; t++) m.prime[t] = t < level ? 0xFF : (uint8_t)(nq + (t - level));
    if ((rc = ntt_launch(ctx, ws.acc, (size_t)batch * 2 * rows, m, true, st)) != FESC_OK) return rc;
    prof_begin(ctx, PF_MODDOWN, st);
    if (bconv_supported(ctx, level))
        moddown_conv_imma_launch(ctx, ws.acc, ws.u, level, batch, ctx->log_n == 16, st);
    else if (N % (256 * KS_VEC) == 0)
        k_moddown_conv<KS_VEC><<<dim3(N / (256 * KS_VEC), batch * 2), 256, 0, st>>>(ws.acc, ws.u, ctx->tabs.d_moddown, ctx->d_pc, N, level, nq, K, ctx->log_n == 16);
    else
        k_moddown_conv<1><<<dim3(gx, batch * 2), 256, 0, st>>>(ws.acc, ws.u, ctx->tabs.d_moddown, ctx->d_pc, N, level, nq, K, ctx->log_n == 16);
    prof_end(ctx, PF_MODDOWN, st);
    m.period = level;
    for (uint32_t i = 0; i < level; i++) m.prime[i] = (uint8_t)i;
    const bool fuse = moddown_fused(ctx, level);
    if (rot_src && !fuse) return fesc_fail(ctx, FESC_EINVAL, "key switch: the permuted addend needs the fused division epilogue");
    if (fuse) {
        NttFinish fin;
        fin.acc = ws.acc, fin.acc_stride = (size_t)2 * rows * N, fin.out = out, fin.out_stride = out_stride, fin.cinv = ctx->tabs.d_moddown->pinvd;
        fin.level = level, fin.acc_rows = rows, fin.add_mask = add_mask;
        fin.rot_src = rot_src, fin.rot_stride = rot_stride, fin.rot_g = rot_g;
        return ntt_launch(ctx, ws.u, (size_t)batch * 2 * level, m, false, st, true, false, &fin);
    }
    if ((rc = ntt_launch(ctx, ws.u, (size_t)batch * 2 * level, m, false, st, ctx->log_n == 16)) != FESC_OK) return rc;
    prof_begin(ctx, PF_MODDOWN, st);
    k_moddown_finish<<<dim3(gx, level, batch * 2), 256, 0, st>>>(ws.acc, ws.u, out, out_stride, ctx->tabs.d_moddown,
                                                                 ctx->d_pc, N, level, K, add_mask);
    prof_end(ctx, PF_MODDOWN, st);
    FESC_CHECK_CUDA(ctx, cudaGetLastError());
    return FESC_OK;
}

// Steps 4-5 for one key.
static int ks_apply(fesc_ctx* ctx, const KsScratch& ws, const EvalKey& key, uint32_t level, uint32_t batch, u64* out,
                    size_t out_stride, int add_mask, cudaStream_t st, u64 g) {
    int rc = ks_inner(ctx, ws, key, level, batch, st, g, 0);
    if (rc != FESC_OK) return rc;
    return ks_moddown(ctx, ws, level, batch, out, out_stride, add_mask, st);
}

// Hybrid key switch of `batch` polynomials d[b] ([level][N], EVAL, contiguous) with scratch
// dcoef (a copy of d, consumed), ext, acc, u.
static int key_switch_chunk(fesc_ctx* ctx, const KsScratch& ws, const EvalKey& key, uint32_t level, uint32_t batch,
                            u64* out, size_t out_stride, int add_mask, cudaStream_t st) {
    int rc = ks_decompose(ctx, ws, level, batch, st);
    if (rc != FESC_OK) return rc;
    return ks_apply(ctx, ws, key, level, batch, out, out_stride, add_mask, st, 0);
}

static OwnRows own_rows(const fesc_ctx* ctx, const KsScratch& ws, uint32_t level) {
    return OwnRows{ws.ext, ctx->alpha, (level + ctx->alpha - 1) / ctx->alpha, level + ctx->n_p, ctx->log_n == 16};
}

size_t ks_scratch_words(const fesc_ctx* ctx, uint32_t level, uint32_t chunk, uint32_t n_ext) {
    const uint32_t beta = (level + ctx->alpha - 1) / ctx->alpha, rows = level + ctx->n_p;
    return (size_t)chunk * ctx->N * ((size_t)level + (size_t)n_ext * beta * rows + 2 * rows + 2 * level);
}
KsScratch ks_scratch_carve(const fesc_ctx* ctx, u64* base, uint32_t level, uint32_t chunk, uint32_t n_ext) {
    const uint32_t beta = (level + ctx->alpha - 1) / ctx->alpha, rows = level + ctx->n_p;
    const size_t N = ctx->N;
    KsScratch ws;
    ws.dcoef = base;
    ws.ext = ws.dcoef + (size_t)chunk * level * N;
    ws.acc = ws.ext + (size_t)n_ext * chunk * beta * rows * N;
    ws.u = ws.acc + (size_t)chunk * 2 * rows * N;
    return ws;
}

uint32_t ks_chunk(const fesc_ctx* ctx, uint32_t batch) {
    // ciphertexts per key-switch pass at N = 2^16 (measured: 16 is 1.5 % faster than 8 on the projection, 3 % on the scan)
    uint32_t c = ctx->log_n == 16 ? 16 : 64;
    static const int e = getenv("FESC_KS_CHUNK") ? atoi(getenv("FESC_KS_CHUNK")) : 0;
    if (e > 0) c = (uint32_t)e;
    return batch < c ? batch : c;
}

// Rotation of `batch` ciphertexts with strides (words) between consecutive inputs / outputs.
// accumulate != 0: the rotated ciphertext is ADDED to what `out` holds.
int rotate_internal(fesc_ctx* ctx, const u64* in, size_t in_stride, u64* out, size_t out_stride, uint32_t batch,
                    uint32_t level, uint32_t key_id, u64* scratch, cudaStream_t st, int accumulate) {
    auto it = ctx->keys.find(key_id);
    if (it == ctx->keys.end() || key_id == FESC_RELIN_KEY_ID)
        return fesc_fail(ctx, FESC_ENOKEY, "rotate: no Galois key " + std::to_string(key_id));
    const uint32_t chunk = ks_chunk(ctx, batch);
    KsScratch ws = ks_scratch_carve(ctx, scratch, level, chunk);
    for (uint32_t b0 = 0; b0 < batch; b0 += chunk) {
        uint32_t nb = batch - b0 < chunk ? batch - b0 : chunk;
        dim3 g((ctx->N + 255) / 256, level, nb);
        const bool fused = moddown_fused(ctx, level);   // then the division's epilogue adds sigma_g(c0) straight from the input
        prof_begin(ctx, PF_AUTOM, st);
        k_autom_ct<<<g, 256, 0, st>>>(in + (size_t)b0 * in_stride, in_stride, fused ? nullptr : out + (size_t)b0 * out_stride, out_stride,
                                      own_rows(ctx, ws, level), ws.dcoef, ctx->log_n, level, it->second.g, ctx->d_pc, accumulate);
        prof_end(ctx, PF_AUTOM, st);
        int rc;
        if (fused) {
            if ((rc = ks_decompose(ctx, ws, level, nb, st)) != FESC_OK) return rc;
            if ((rc = ks_inner(ctx, ws, it->second, level, nb, st, 0, 0)) != FESC_OK) return rc;
            rc = ks_moddown(ctx, ws, level, nb, out + (size_t)b0 * out_stride, out_stride, accumulate ? 3 : 0, st,
                            in + (size_t)b0 * in_stride, in_stride, it->second.g);
        } else {
            rc = key_switch_chunk(ctx, ws, it->second, level, nb, out + (size_t)b0 * out_stride, out_stride,
                                  accumulate ? 3 : 1, st);
        }
        if (rc != FESC_OK) return rc;
    }
    return FESC_OK;
}

// c0 of every ciphertext through the Galois permutation into out[b][0]; with g == 0, c1 copied to d and dcoef
__global__ void __launch_bounds__(256) k_hoist_prepare(const u64* __restrict__ in, size_t in_stride, u64* __restrict__ out0,
                                                       size_t out_stride, OwnRows d, u64* __restrict__ dcoef,
                                                       uint32_t log_n, uint32_t level, u64 g,
                                                       const PrimeConst* __restrict__ pcs) {
    const uint32_t N = 1u << log_n;
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t l = blockIdx.y, b = blockIdx.z;
    if (t >= N) return;
    const u64* ib = in + (size_t)b * in_stride;
    if (g) {
        if (galois_src(t, log_n, g) >= N || !DBG_REGION(ib + (size_t)l * N, N * sizeof(u64)) ||
            !DBG_REGION(out0 + (size_t)b * out_stride + (size_t)l * N, N * sizeof(u64)))
            return;
        out0[(size_t)b * out_stride + (size_t)l * N + t] = ib[(size_t)l * N + galois_src(t, log_n, g)];
    } else {
        if (!DBG_REGION(ib + ((size_t)level + l) * N, N * sizeof(u64)) || !DBG_REGION(d.ext + own_index(d, b, l, N), N * sizeof(u64)) ||
            !DBG_REGION(dcoef + ((size_t)b * level + l) * N, N * sizeof(u64)))
            return;
        const u64 v = ib[((size_t)level + l) * N + t];
        d.ext[own_index(d, b, l, N) + t] = own_word(d, v, pcs[l]);
        dcoef[((size_t)b * level + l) * N + t] = v;
    }
}

// sum_p rot(acc[b][p], key n = key_base + p) for p = 1..n_terms-1 ADDED into acc[b][0], with one division by P
// per ciphertext: the inner products of all p are summed on the extended basis first.  acc holds `batch` groups of
// n_terms ciphertexts (ct_words each, group stride n_terms * ct_words).
int giant_sum_deferred_internal(fesc_ctx* ctx, u64* acc, uint32_t n_terms, size_t ct_words, uint32_t batch,
                                uint32_t level, uint32_t key_base, u64* scratch, cudaStream_t st) {
    if (n_terms < 2) return FESC_OK;
    for (uint32_t p = 1; p < n_terms; p++)
        if (!ctx->keys.count(key_base + p) || key_base + p == FESC_RELIN_KEY_ID)
            return fesc_fail(ctx, FESC_ENOKEY, "giant steps: no Galois key " + std::to_string(key_base + p));
    const uint32_t chunk = ks_chunk(ctx, batch), n_ext = giant_ext_buffers(n_terms);
    KsScratch ws = ks_scratch_carve(ctx, scratch, level, chunk, n_ext);
    const size_t stride = (size_t)n_terms * ct_words;
    const size_t ext_words = (size_t)chunk * ((level + ctx->alpha - 1) / ctx->alpha) * (level + ctx->n_p) * ctx->N;
    for (uint32_t b0 = 0; b0 < batch; b0 += chunk) {
        const uint32_t nb = batch - b0 < chunk ? batch - b0 : chunk;
        dim3 g((ctx->N + 255) / 256, level, nb);
        u64* base = acc + (size_t)b0 * stride;
        // up to n_ext terms are rotated and converted side by side, then one inner-product pass sums them: the
        // accumulators on the extended basis are read and written once per pass instead of once per term
        for (uint32_t p0 = 1; p0 < n_terms; p0 += n_ext) {
            const uint32_t np = n_terms - p0 < n_ext ? n_terms - p0 : n_ext;
            InnerSrcs S;
            S.n = np;
            for (uint32_t s = 0; s < np; s++) {
                const EvalKey& key = ctx->keys[key_base + p0 + s];
                KsScratch wss = ws;
                wss.ext = ws.ext + (size_t)s * ext_words;
                prof_begin(ctx, PF_AUTOM, st);
                k_autom_ct<<<g, 256, 0, st>>>(base + (size_t)(p0 + s) * ct_words, stride, base, stride, own_rows(ctx, wss, level),
                                              wss.dcoef, ctx->log_n, level, key.g, ctx->d_pc, 1);
                prof_end(ctx, PF_AUTOM, st);
                int rc = ks_decompose(ctx, wss, level, nb, st);
                if (rc != FESC_OK) return rc;
                S.s[s] = InnerSrc{wss.ext, key.d_key, 0};
            }
            int rc = ks_inner_multi(ctx, ws, S, level, nb, st, p0 > 1);
            if (rc != FESC_OK) return rc;
        }
        int rc = ks_moddown(ctx, ws, level, nb, base, stride, 3, st);
        if (rc != FESC_OK) return rc;
    }
    return FESC_OK;
}

// Hoisted rotations: every ciphertext of the batch is decomposed once and rotated by each of the n_keys
// keys.  Output k of ciphertext b goes to out + k*key_stride + b*out_stride.
int rotate_hoisted_internal(fesc_ctx* ctx, const u64* in, size_t in_stride, u64* out, size_t out_stride,
                            size_t key_stride, uint32_t batch, uint32_t level, const uint32_t* key_ids, uint32_t n_keys,
                            u64* scratch, cudaStream_t st) {
    for (uint32_t k = 0; k < n_keys; k++)
        if (!ctx->keys.count(key_ids[k]) || key_ids[k] == FESC_RELIN_KEY_ID)
            return fesc_fail(ctx, FESC_ENOKEY, "rotate_hoisted: no Galois key " + std::to_string(key_ids[k]));
    const uint32_t chunk = ks_chunk(ctx, batch);
    KsScratch ws = ks_scratch_carve(ctx, scratch, level, chunk);
    for (uint32_t b0 = 0; b0 < batch; b0 += chunk) {
        const uint32_t nb = batch - b0 < chunk ? batch - b0 : chunk;
        dim3 g((ctx->N + 255) / 256, level, nb);
        const u64* ib = in + (size_t)b0 * in_stride;
        prof_begin(ctx, PF_AUTOM, st);
        k_hoist_prepare<<<g, 256, 0, st>>>(ib, in_stride, nullptr, 0, own_rows(ctx, ws, level), ws.dcoef, ctx->log_n, level, 0, ctx->d_pc);
        prof_end(ctx, PF_AUTOM, st);
        int rc = ks_decompose(ctx, ws, level, nb, st);
        if (rc != FESC_OK) return rc;
        for (uint32_t k = 0; k < n_keys; k++) {
            const EvalKey& key = ctx->keys[key_ids[k]];
            u64* ob = out + (size_t)k * key_stride + (size_t)b0 * out_stride;
            if (moddown_fused(ctx, level)) {     // sigma_g(c0) is added by the division's epilogue, straight from the input
                if ((rc = ks_inner(ctx, ws, key, level, nb, st, key.g, 0)) != FESC_OK) return rc;
                if ((rc = ks_moddown(ctx, ws, level, nb, ob, out_stride, 0, st, ib, in_stride, key.g)) != FESC_OK) return rc;
                continue;
            }
            prof_begin(ctx, PF_AUTOM, st);
            k_hoist_prepare<<<g, 256, 0, st>>>(ib, in_stride, ob, out_stride, OwnRows{nullptr, 1, 1, 1, 0}, nullptr, ctx->log_n, level, key.g, ctx->d_pc);
            prof_end(ctx, PF_AUTOM, st);
            rc = ks_apply(ctx, ws, key, level, nb, ob, out_stride, 1, st, key.g);
            if (rc != FESC_OK) return rc;
        }
    }
    return FESC_OK;
}

// out = in + sum_k rot_k(in): c0 and the Galois images of c0 are summed here, c1 is copied; the key-switch part
// is added by the division step.
struct GaloisSet {
    u64 g[8];
    uint32_t n;
};
__global__ void __launch_bounds__(256) k_rotsum_prepare(const u64* __restrict__ in, size_t in_stride, u64* __restrict__ out,
                                                        size_t out_stride, uint32_t log_n, uint32_t level, GaloisSet gs,
                                                        const PrimeConst* __restrict__ pcs) {
    const uint32_t N = 1u << log_n;
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t l = blockIdx.y, b = blockIdx.z;
    if (t >= N) return;
    const u64* ib = in + (size_t)b * in_stride;
    u64* ob = out + (size_t)b * out_stride;
    const u64 q = pcs[l].q;
    for (int p = 0; p < 2; p++)
        if (!DBG_REGION(ib + ((size_t)p * level + l) * N, N * sizeof(u64)) || !DBG_REGION(ob + ((size_t)p * level + l) * N, N * sizeof(u64)))
            return;
    u64 v = ib[(size_t)l * N + t];
    for (uint32_t k = 0; k < gs.n; k++) v = addmod(v, ib[(size_t)l * N + galois_src(t, log_n, gs.g[k])], q);
    ob[(size_t)l * N + t] = v;
    ob[((size_t)level + l) * N + t] = ib[((size_t)level + l) * N + t];
}

// out[b] = in[b] + sum_k rot(in[b], key k): one decomposition per ciphertext, the inner products of all keys summed
// on the extended basis, one division by P (in and out must not overlap; at most 8 keys).
int rotate_sum_hoisted_internal(fesc_ctx* ctx, const u64* in, size_t in_stride, u64* out, size_t out_stride,
                                uint32_t batch, uint32_t level, const uint32_t* key_ids, uint32_t n_keys, u64* scratch,
                                cudaStream_t st) {
    if (n_keys == 0 || n_keys > 8) return fesc_fail(ctx, FESC_EINVAL, "rotate_sum_hoisted: 1 to 8 keys");
    GaloisSet gs;
    gs.n = n_keys;
    for (uint32_t k = 0; k < n_keys; k++) {
        if (!ctx->keys.count(key_ids[k]) || key_ids[k] == FESC_RELIN_KEY_ID)
            return fesc_fail(ctx, FESC_ENOKEY, "rotate_sum_hoisted: no Galois key " + std::to_string(key_ids[k]));
        gs.g[k] = ctx->keys[key_ids[k]].g;
    }
    const uint32_t chunk = ks_chunk(ctx, batch);
    KsScratch ws = ks_scratch_carve(ctx, scratch, level, chunk);
    for (uint32_t b0 = 0; b0 < batch; b0 += chunk) {
        const uint32_t nb = batch - b0 < chunk ? batch - b0 : chunk;
        dim3 g((ctx->N + 255) / 256, level, nb);
        const u64* ib = in + (size_t)b0 * in_stride;
        u64* ob = out + (size_t)b0 * out_stride;
        prof_begin(ctx, PF_AUTOM, st);
        k_hoist_prepare<<<g, 256, 0, st>>>(ib, in_stride, nullptr, 0, own_rows(ctx, ws, level), ws.dcoef, ctx->log_n, level, 0, ctx->d_pc);
        k_rotsum_prepare<<<g, 256, 0, st>>>(ib, in_stride, ob, out_stride, ctx->log_n, level, gs, ctx->d_pc);
        prof_end(ctx, PF_AUTOM, st, 2);
        int rc = ks_decompose(ctx, ws, level, nb, st);
        if (rc != FESC_OK) return rc;
        InnerSrcs S;                                   // one converted polynomial, read through every key's permutation
        S.n = n_keys;
        for (uint32_t k = 0; k < n_keys; k++) S.s[k] = InnerSrc{ws.ext, ctx->keys[key_ids[k]].d_key, gs.g[k]};
        if ((rc = ks_inner_multi(ctx, ws, S, level, nb, st, 0)) != FESC_OK) return rc;
        if ((rc = ks_moddown(ctx, ws, level, nb, ob, out_stride, 3, st)) != FESC_OK) return rc;
    }
    return FESC_OK;
}

extern "C" int fesc_rotate_sum_hoisted(fesc_ctx* ctx, const uint64_t* d_in, uint64_t* d_out, uint32_t batch,
                                       uint32_t n_limbs, const uint32_t* key_ids, uint32_t n_keys, void* stream) {
    if (!ctx || !d_in || !d_out || !key_ids || d_in == d_out) return FESC_EINVAL;
    if (n_limbs == 0 || n_limbs > ctx->n_q) return fesc_fail(ctx, FESC_ELEVEL, "rotate_sum_hoisted: level out of range");
    if (batch == 0) return FESC_OK;
    u64* scratch;
    int rc = ctx_scratch(ctx, ks_scratch_words(ctx, n_limbs, ks_chunk(ctx, batch)) * sizeof(u64), &scratch);
    if (rc != FESC_OK) return rc;
    const size_t stride = (size_t)2 * n_limbs * ctx->N;
    return rotate_sum_hoisted_internal(ctx, (const u64*)d_in, stride, (u64*)d_out, stride, batch, n_limbs, key_ids,
                                       n_keys, scratch, (cudaStream_t)stream);
}

extern "C" int fesc_rotate_hoisted(fesc_ctx* ctx, const uint64_t* d_in, uint64_t* d_out, uint32_t batch,
                                   uint32_t n_limbs, const uint32_t* key_ids, uint32_t n_keys, void* stream) {
    if (!ctx || !d_in || !d_out || (!key_ids && n_keys) || d_in == d_out) return FESC_EINVAL;
    if (n_limbs == 0 || n_limbs > ctx->n_q) return fesc_fail(ctx, FESC_ELEVEL, "rotate_hoisted: level out of range");
    if (batch == 0 || n_keys == 0) return FESC_OK;
    u64* scratch;
    int rc = ctx_scratch(ctx, ks_scratch_words(ctx, n_limbs, ks_chunk(ctx, batch)) * sizeof(u64), &scratch);
    if (rc != FESC_OK) return rc;
    const size_t stride = (size_t)2 * n_limbs * ctx->N;
    return rotate_hoisted_internal(ctx, (const u64*)d_in, stride, (u64*)d_out, stride, (size_t)batch * stride, batch,
                                   n_limbs, key_ids, n_keys, scratch, (cudaStream_t)stream);
}

extern "C" int fesc_rotate(fesc_ctx* ctx, const uint64_t* d_in, uint64_t* d_out, uint32_t batch, uint32_t n_limbs,
                           uint32_t key_id, void* stream) {
    if (!ctx || !d_in || !d_out || d_in == d_out) return FESC_EINVAL;      // the input is read while the output is written
    if (n_limbs == 0 || n_limbs > ctx->n_q) return fesc_fail(ctx, FESC_ELEVEL, "rotate: level out of range");
    if (batch == 0) return FESC_OK;
    u64* scratch;
    int rc = ctx_scratch(ctx, ks_scratch_words(ctx, n_limbs, ks_chunk(ctx, batch)) * sizeof(u64), &scratch);
    if (rc != FESC_OK) return rc;
    const size_t stride = (size_t)2 * n_limbs * ctx->N;
    return rotate_internal(ctx, (const u64*)d_in, stride, (u64*)d_out, stride, batch, n_limbs, key_id, scratch,
                           (cudaStream_t)stream, 0);
}

// ---------------------------------------------------------------------------------------
// Rescale
// ---------------------------------------------------------------------------------------
// gather the last limb of every polynomial into r[b*2+p][N]
__global__ void __launch_bounds__(256) k_take_last(const u64* __restrict__ in, size_t in_stride, u64* __restrict__ r,
                                                   uint32_t N, uint32_t level) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t bp = blockIdx.y;
    if (c >= N) return;
    if (!DBG_REGION(r + (size_t)bp * N, N * sizeof(u64)) ||
        !DBG_REGION(in + (size_t)(bp >> 1) * in_stride + ((size_t)(bp & 1) * level + level - 1) * N, N * sizeof(u64)))
        return;
    r[(size_t)bp * N + c] = in[(size_t)(bp >> 1) * in_stride + ((size_t)(bp & 1) * level + level - 1) * N + c];
}
// out[b][p][i] = centred(r) mod q_i  (COEFF)
__global__ void __launch_bounds__(256) k_rescale_conv(const u64* __restrict__ r, u64* __restrict__ out, size_t out_stride,
                                                      const RescaleTab* __restrict__ tab,
                                                      const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t i = blockIdx.y, bp = blockIdx.z;
    if (c >= N) return;
    if (!DBG_REGION(r + (size_t)bp * N, N * sizeof(u64)) || !DBG_REGION(tab, sizeof(RescaleTab)) ||
        !DBG_REGION(out + (size_t)(bp >> 1) * out_stride + ((size_t)(bp & 1) * (level - 1) + i) * N, N * sizeof(u64)))
        return;
    const u64 v = r[(size_t)bp * N + c];
    const PrimeConst pc = pcs[i];
    u64 w = v - mulhi(v, pc.mu) * pc.q;   // v mod q_i in [0, 2q)
    w = csub(w, pc.q);
    if (v > tab->half) w = submod(w, tab->wrap[i], pc.q);
    out[(size_t)(bp >> 1) * out_stride + ((size_t)(bp & 1) * (level - 1) + i) * N + c] = w;
}
// out = (in - out) * q_last^-1
__global__ void __launch_bounds__(256) k_rescale_finish(const u64* __restrict__ in, size_t in_stride,
                                                        u64* __restrict__ out, size_t out_stride,
                                                        const RescaleTab* __restrict__ tab,
                                                        const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t i = blockIdx.y, bp = blockIdx.z;
    if (c >= N) return;
    const u64 q = pcs[i].q;
    u64* o = out + (size_t)(bp >> 1) * out_stride + ((size_t)(bp & 1) * (level - 1) + i) * N + c;
    if (!DBG_REGION(o - c, N * sizeof(u64)) || !DBG_REGION(tab, sizeof(RescaleTab)) ||
        !DBG_REGION(in + (size_t)(bp >> 1) * in_stride + ((size_t)(bp & 1) * level + i) * N, N * sizeof(u64)))
        return;
    u64 x = in[(size_t)(bp >> 1) * in_stride + ((size_t)(bp & 1) * level + i) * N + c];
    *o = shoup(submod(x, *o, q), tab->qinv[i], tab->qinvs[i], q);
}

// out must be a contiguous batch [batch][2][level-1][N]; scratch holds batch*2*N words.
int rescale_internal(fesc_ctx* ctx, const u64* in, size_t in_stride, u64* out, uint32_t batch, uint32_t level,
                     u64* scratch, cudaStream_t st) {
    const uint32_t N = ctx->N, gx = (N + 255) / 256;
    const size_t out_stride = (size_t)2 * (level - 1) * N;
    const RescaleTab* tab = ctx->tabs.d_rescale + level;
    int rc;
    for (uint32_t b0 = 0; b0 < batch; b0 += 16384) {
        uint32_t nb = batch - b0 < 16384 ? batch - b0 : 16384;
        const u64* ib = in + (size_t)b0 * in_stride;
        u64* ob = out + (size_t)b0 * out_stride;
        prof_begin(ctx, PF_RESCALE, st);
        k_take_last<<<dim3(gx, nb * 2), 256, 0, st>>>(ib, in_stride, scratch, N, level);
        prof_end(ctx, PF_RESCALE, st);
        RowMap m;
        m.period = 1;
        m.prime[0] = (uint8_t)(level - 1);
        if ((rc = ntt_launch(ctx, scratch, (size_t)nb * 2, m, true, st)) != FESC_OK) return rc;
        prof_begin(ctx, PF_RESCALE, st);
        k_rescale_conv<<<dim3(gx, level - 1, nb * 2), 256, 0, st>>>(scratch, ob, out_stride, tab, ctx->d_pc, N, level);
        prof_end(ctx, PF_RESCALE, st);
        m.period = level - 1;
        for (uint32_t i = 0; i + 1 < level; i++) m.prime[i] = (uint8_t)i;
        // N = 2^16, FP64 rows: the last pass of the transform stores (in - u) * q_last^-1 itself
        bool fuse = ctx->log_n == 16;
        for (uint32_t i = 0; i + 1 < level; i++) fuse = fuse && ctx->q[i] < FESC_FP_LIMIT;
        if (fuse) {
            NttFinish fin;
            fin.acc = ib, fin.acc_stride = in_stride, fin.out = ob, fin.out_stride = out_stride, fin.cinv = tab->qinvd;
            fin.level = level - 1, fin.acc_rows = level, fin.add_mask = 0;
            if ((rc = ntt_launch(ctx, ob, (size_t)nb * 2 * (level - 1), m, false, st, false, false, &fin)) != FESC_OK) return rc;
            continue;
        }
        if ((rc = ntt_launch(ctx, ob, (size_t)nb * 2 * (level - 1), m, false, st)) != FESC_OK) return rc;
        prof_begin(ctx, PF_RESCALE, st);
        k_rescale_finish<<<dim3(gx, level - 1, nb * 2), 256, 0, st>>>(ib, in_stride, ob, out_stride, tab, ctx->d_pc, N,
                                                                    level);
        prof_end(ctx, PF_RESCALE, st);
    }
    FESC_CHECK_CUDA(ctx, cudaGetLastError());
    return FESC_OK;
}

extern "C" int fesc_rescale(fesc_ctx* ctx, const uint64_t* d_in, uint64_t* d_out, uint32_t batch, uint32_t n_limbs,
                            void* stream) {
    if (!ctx || !d_in || !d_out) return FESC_EINVAL;
    if (n_limbs < 2 || n_limbs > ctx->n_q) return fesc_fail(ctx, FESC_ELEVEL, "rescale: level out of range");
    if (batch == 0) return FESC_OK;
    u64* scratch;
    uint32_t nb = batch < 16384 ? batch : 16384;
    int rc = ctx_scratch(ctx, (size_t)nb * 2 * ctx->N * sizeof(u64), &scratch);
    if (rc != FESC_OK) return rc;
    return rescale_internal(ctx, (const u64*)d_in, (size_t)2 * n_limbs * ctx->N, (u64*)d_out, batch, n_limbs, scratch,
                            (cudaStream_t)stream);
}

// ---------------------------------------------------------------------------------------
// ct x ct: tensor product, then relinearisation of d2
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_tensor(const u64* __restrict__ a, size_t a_stride, const u64* __restrict__ bb,
                                                size_t b_stride, u64* __restrict__ out, size_t out_stride,
                                                OwnRows d, u64* __restrict__ dcoef,
                                                const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t l = blockIdx.y, b = blockIdx.z;
    if (c >= N) return;
    const PrimeConst pc = pcs[l];
    const size_t poly = (size_t)level * N, o = (size_t)l * N + c;
    for (int p = 0; p < 2; p++)
        if (!DBG_REGION(a + b * a_stride + p * poly + o - c, N * sizeof(u64)) || !DBG_REGION(bb + b * b_stride + p * poly + o - c, N * sizeof(u64)) ||
            !DBG_REGION(out + b * out_stride + p * poly + o - c, N * sizeof(u64)))
            return;
    if (!DBG_REGION(d.ext + own_index(d, b, l, N), N * sizeof(u64)) || !DBG_REGION(dcoef + ((size_t)b * level + l) * N, N * sizeof(u64))) return;
    const u64 a0 = a[b * a_stride + o], a1 = a[b * a_stride + poly + o];
    const u64 b0 = bb[b * b_stride + o], b1 = bb[b * b_stride + poly + o];
    out[b * out_stride + o] = mulmod(a0, b0, pc);
    acc128 s{0, 0};
    mac128(s, a0, b1);
    mac128(s, a1, b0);
    out[b * out_stride + poly + o] = reduce128(s.hi, s.lo, pc);
    const u64 d2 = mulmod(a1, b1, pc);
    d.ext[own_index(d, b, l, N) + c] = own_word(d, d2, pc);
    dcoef[((size_t)b * level + l) * N + c] = d2;
}

int ctmul_internal(fesc_ctx* ctx, const u64* a, size_t a_stride, const u64* b, size_t b_stride, u64* out,
                   size_t out_stride, uint32_t batch, uint32_t level, u64* scratch, cudaStream_t st) {
    const EvalKey& key = ctx->keys[FESC_RELIN_KEY_ID];
    const uint32_t chunk = ks_chunk(ctx, batch);
    KsScratch ws = ks_scratch_carve(ctx, scratch, level, chunk);
    for (uint32_t b0 = 0; b0 < batch; b0 += chunk) {
        uint32_t nb = batch - b0 < chunk ? batch - b0 : chunk;
        dim3 g((ctx->N + 255) / 256, level, nb);
        prof_begin(ctx, PF_POINTWISE, st);
        k_tensor<<<g, 256, 0, st>>>(a + (size_t)b0 * a_stride, a_stride, b + (size_t)b0 * b_stride, b_stride,
                                    out + (size_t)b0 * out_stride, out_stride, own_rows(ctx, ws, level), ws.dcoef, ctx->d_pc, ctx->N, level);
        prof_end(ctx, PF_POINTWISE, st);
        int rc = key_switch_chunk(ctx, ws, key, level, nb, out + (size_t)b0 * out_stride, out_stride, 3, st);
        if (rc != FESC_OK) return rc;
    }
    return FESC_OK;
}

extern "C" int fesc_ct_ct_mul(fesc_ctx* ctx, const uint64_t* d_a, const uint64_t* d_b, uint64_t* d_out, uint32_t batch,
                              uint32_t n_limbs, void* stream) {
    if (!ctx || !d_a || !d_b || !d_out) return FESC_EINVAL;
    if (n_limbs == 0 || n_limbs > ctx->n_q) return fesc_fail(ctx, FESC_ELEVEL, "ct_ct_mul: level out of range");
    if (batch == 0) return FESC_OK;
    u64* scratch;
    int rc = ctx_scratch(ctx, ks_scratch_words(ctx, n_limbs, ks_chunk(ctx, batch)) * sizeof(u64), &scratch);
    if (rc != FESC_OK) return rc;
    const size_t stride = (size_t)2 * n_limbs * ctx->N;
    return ctmul_internal(ctx, (const u64*)d_a, stride, (const u64*)d_b, stride, (u64*)d_out, stride, batch, n_limbs,
                          scratch, (cudaStream_t)stream);
}
