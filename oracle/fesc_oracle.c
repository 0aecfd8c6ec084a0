/*
 * CPU oracle primitives for the RNS-CKKS linear hot path (TEST INFRASTRUCTURE).
 *
 * This file is the slow, plain checker that the CUDA library is compared
 * against.  It is test infrastructure only: nothing in the product path may
 * call it, and it shares no code, header, table or constant with the CUDA
 * sources.  Every modular product is a 128-bit product followed by `%`.
 *
 * What is here: limb-wise negacyclic NTT / inverse NTT, pointwise modular
 * arithmetic, the Galois permutation in evaluation order, fast RNS basis
 * conversion (the approximate, uncorrected form used by hybrid key switching
 * and by rounding division), and the counter-based samplers the key generator
 * draws from.  The compositions (key switch, rotation, rescale, ct x ct, BSGS
 * projection, scan-contract) are written in Python on top of these, in the
 * order the paper gives (oracle/ckks.py).
 *
 * The paper (Sec. 5.1, Table "CKKS primitives") treats add / ptmul / ctmul /
 * rot / conj as black boxes, so the constructions below are the standard
 * RNS-CKKS ones with these conventions:
 *   - residues are canonical, in [0, q);
 *   - psi is the SMALLEST primitive 2N-th root of unity mod q;
 *   - evaluation order: EVAL[t] = sum_i COEFF[i] * psi^((2*brev(t)+1)*i) mod q.
 *
 * The transform is computed as a twist by psi^i followed by a textbook cyclic
 * decimation-in-frequency FFT over Z_q with omega = psi^2 (natural order in,
 * bit-reversed order out): X[k] = sum_i (a_i psi^i) omega^(ik) lands at index
 * brev(k), which is exactly the order above.  tests/ pins it against the
 * O(N^2) sum.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef uint64_t u64;
typedef unsigned __int128 u128;

static inline u64 mulmod(u64 a, u64 b, u64 q) { return (u64)((u128)a * b % q); }
static inline u64 addmod(u64 a, u64 b, u64 q) { u64 s = a + b; return s >= q ? s - q : s; }
static inline u64 submod(u64 a, u64 b, u64 q) { return a >= b ? a - b : a + q - b; }

static u64 powmod(u64 a, u64 e, u64 q) {
    u64 r = 1 % q;
    a %= q;
    while (e) {
        if (e & 1) r = mulmod(r, a, q);
        a = mulmod(a, a, q);
        e >>= 1;
    }
    return r;
}

u64 orc_powmod(u64 a, u64 e, u64 q) { return powmod(a, e, q); }
u64 orc_invmod(u64 a, u64 q) { return powmod(a, q - 2, q); } /* q prime */

static uint32_t brev(uint32_t x, uint32_t bits) {
    uint32_t r = 0;
    for (uint32_t i = 0; i < bits; i++) { r = (r << 1) | (x & 1); x >>= 1; }
    return r;
}

/* Smallest primitive 2N-th root of unity mod q (q prime, q = 1 mod 2N). 0 on failure. */
u64 orc_min_psi(u64 q, uint32_t logN) {
    u64 N = 1ull << logN, twoN = 2 * N;
    if ((q - 1) % twoN) return 0;
    u64 x = 0;
    for (u64 g = 2; g < 1000; g++) {
        u64 c = powmod(g, (q - 1) / twoN, q);
        if (powmod(c, N, q) == q - 1) { x = c; break; }
    }
    if (!x) return 0;
    /* all primitive 2N-th roots are the odd powers of x */
    u64 x2 = mulmod(x, x, q), cur = x, best = x;
    for (u64 i = 0; i < N; i++) {
        if (cur < best) best = cur;
        cur = mulmod(cur, x2, q);
    }
    return best;
}

/* Forward transform of k limbs; limb i is a[i*N .. (i+1)*N) modulo q[i]. */
void orc_ntt(u64* a, const u64* q, uint32_t k, uint32_t logN) {
    const u64 N = 1ull << logN;
#pragma omp parallel for schedule(dynamic)
    for (uint32_t l = 0; l < k; l++) {
        u64* x = a + (size_t)l * N;
        const u64 p = q[l];
        const u64 psi = orc_min_psi(p, logN);
        const u64 omega = mulmod(psi, psi, p);
        u64* wpow = (u64*)malloc(sizeof(u64) * N); /* omega^i, i < N/2 used */
        u64 t = 1;
        for (u64 i = 0; i < N; i++) { x[i] = mulmod(x[i], t, p); t = mulmod(t, psi, p); }
        t = 1;
        for (u64 i = 0; i < N / 2; i++) { wpow[i] = t; t = mulmod(t, omega, p); }
        for (u64 len = N / 2; len >= 1; len >>= 1) {
            const u64 step = N / (2 * len);
            for (u64 s = 0; s < N; s += 2 * len)
                for (u64 j = 0; j < len; j++) {
                    u64 u = x[s + j], v = x[s + j + len];
                    x[s + j] = addmod(u, v, p);
                    x[s + j + len] = mulmod(submod(u, v, p), wpow[j * step], p);
                }
        }
        free(wpow);
    }
}

/* Inverse of orc_ntt (includes the factor N^-1). */
void orc_intt(u64* a, const u64* q, uint32_t k, uint32_t logN) {
    const u64 N = 1ull << logN;
#pragma omp parallel for schedule(dynamic)
    for (uint32_t l = 0; l < k; l++) {
        u64* x = a + (size_t)l * N;
        const u64 p = q[l];
        const u64 psi = orc_min_psi(p, logN);
        const u64 ipsi = orc_invmod(psi, p);
        const u64 iomega = mulmod(ipsi, ipsi, p);
        u64* wpow = (u64*)malloc(sizeof(u64) * N);
        u64 t = 1;
        for (u64 i = 0; i < N / 2; i++) { wpow[i] = t; t = mulmod(t, iomega, p); }
        /* decimation in time: bit-reversed in, natural out */
        for (u64 len = 1; len < N; len <<= 1) {
            const u64 step = N / (2 * len);
            for (u64 s = 0; s < N; s += 2 * len)
                for (u64 j = 0; j < len; j++) {
                    u64 u = x[s + j], v = mulmod(x[s + j + len], wpow[j * step], p);
                    x[s + j] = addmod(u, v, p);
                    x[s + j + len] = submod(u, v, p);
                }
        }
        const u64 ninv = orc_invmod(N % p, p);
        t = ninv;
        for (u64 i = 0; i < N; i++) { x[i] = mulmod(x[i], t, p); t = mulmod(t, ipsi, p); }
        free(wpow);
    }
}

/* Direct O(N^2) evaluation of the definition, for pins on small N. */
void orc_ntt_direct(const u64* a, u64* out, u64 q, uint32_t logN) {
    const u64 N = 1ull << logN;
    const u64 psi = orc_min_psi(q, logN);
    for (u64 t = 0; t < N; t++) {
        u64 e = 2 * (u64)brev((uint32_t)t, logN) + 1;
        u64 root = powmod(psi, e, q), cur = 1, acc = 0;
        for (u64 i = 0; i < N; i++) {
            acc = addmod(acc, mulmod(a[i] % q, cur, q), q);
            cur = mulmod(cur, root, q);
        }
        out[t] = acc;
    }
}

/* ---- pointwise, k limbs of n entries, limb i modulo q[i] ---- */
void orc_mul(const u64* a, const u64* b, u64* out, const u64* q, uint32_t k, u64 n) {
#pragma omp parallel for
    for (uint32_t l = 0; l < k; l++)
        for (u64 i = 0; i < n; i++) out[l * n + i] = mulmod(a[l * n + i], b[l * n + i], q[l]);
}
/* acc += a*b */
void orc_muladd(const u64* a, const u64* b, u64* acc, const u64* q, uint32_t k, u64 n) {
#pragma omp parallel for
    for (uint32_t l = 0; l < k; l++)
        for (u64 i = 0; i < n; i++)
            acc[l * n + i] = addmod(acc[l * n + i], mulmod(a[l * n + i], b[l * n + i], q[l]), q[l]);
}
void orc_add(const u64* a, const u64* b, u64* out, const u64* q, uint32_t k, u64 n) {
#pragma omp parallel for
    for (uint32_t l = 0; l < k; l++)
        for (u64 i = 0; i < n; i++) out[l * n + i] = addmod(a[l * n + i], b[l * n + i], q[l]);
}
void orc_sub(const u64* a, const u64* b, u64* out, const u64* q, uint32_t k, u64 n) {
#pragma omp parallel for
    for (uint32_t l = 0; l < k; l++)
        for (u64 i = 0; i < n; i++) out[l * n + i] = submod(a[l * n + i], b[l * n + i], q[l]);
}
/* out = a * c[l] (one scalar per limb, already reduced) */
void orc_mul_scalar(const u64* a, const u64* c, u64* out, const u64* q, uint32_t k, u64 n) {
#pragma omp parallel for
    for (uint32_t l = 0; l < k; l++)
        for (u64 i = 0; i < n; i++) out[l * n + i] = mulmod(a[l * n + i], c[l] % q[l], q[l]);
}
/* out = a + c[l] */
void orc_add_scalar(const u64* a, const u64* c, u64* out, const u64* q, uint32_t k, u64 n) {
#pragma omp parallel for
    for (uint32_t l = 0; l < k; l++)
        for (u64 i = 0; i < n; i++) out[l * n + i] = addmod(a[l * n + i], c[l] % q[l], q[l]);
}

/* ---- Galois automorphism a(X) -> a(X^g), g odd ---- */
/* coefficient form: coefficient i moves to i*g mod 2N, negated when that is >= N */
void orc_autom_coeff(const u64* a, u64* out, const u64* q, uint32_t k, uint32_t logN, u64 g) {
    const u64 N = 1ull << logN, mask = 2 * N - 1;
    for (uint32_t l = 0; l < k; l++)
        for (u64 i = 0; i < N; i++) {
            u64 j = (i * g) & mask;
            u64 v = a[l * N + i];
            if (j >= N) out[l * N + (j - N)] = v ? q[l] - v : 0;
            else out[l * N + j] = v;
        }
}
/* evaluation form (bit-reversed order): out[t] = in[pi_g(t)], where slot t holds the
 * value at psi^(2 brev(t)+1) and sigma_g(a) evaluated there is a at psi^((2 brev(t)+1) g) */
void orc_autom_eval(const u64* a, u64* out, uint32_t k, uint32_t logN, u64 g) {
    const u64 N = 1ull << logN, mask = 2 * N - 1;
#pragma omp parallel for
    for (uint32_t l = 0; l < k; l++)
        for (u64 t = 0; t < N; t++) {
            u64 e = ((2 * (u64)brev((uint32_t)t, logN) + 1) * g) & mask;
            u64 src = brev((uint32_t)((e - 1) / 2), logN);
            out[l * N + t] = a[l * N + src];
        }
}

/* ---- fast (uncorrected) basis conversion ----
 * in : ks limbs modulo src[0..ks), each of n entries
 * out: kd limbs modulo dst[0..kd)
 * With S = prod src, S_i = S/src_i:  y_i = in_i * (S_i^-1 mod src_i) mod src_i,
 * out_t = sum_i y_i * (S_i mod dst_t) mod dst_t  (no correction term).
 * centred == 0: y_i is the canonical representative in [0, src_i); the value
 *   represented is [x]_S + u*S with an integer 0 <= u < ks   (used by ModUp).
 * centred != 0: y_i is the representative in [-(src_i-1)/2, (src_i-1)/2]; the value
 *   represented is x' = x (mod S) with |x'| < ks*S/2, so that (c - x')/S differs from
 *   c/S by sum_i y_i/src_i, a zero-mean quantity   (used by the divisions by P and by
 *   the dropped prime; with ks == 1 it is the exact centred remainder). */
void orc_fast_conv(const u64* in, const u64* src, uint32_t ks, const u64* dst, uint32_t kd,
                   u64* out, u64 n, int centred) {
    u64* y = (u64*)malloc(sizeof(u64) * (size_t)ks * n);
    for (uint32_t i = 0; i < ks; i++) {
        u64 si = 1;
        for (uint32_t j = 0; j < ks; j++)
            if (j != i) si = mulmod(si, src[j] % src[i], src[i]);
        u64 inv = orc_invmod(si, src[i]);
#pragma omp parallel for
        for (u64 c = 0; c < n; c++) y[(size_t)i * n + c] = mulmod(in[(size_t)i * n + c], inv, src[i]);
    }
#pragma omp parallel for
    for (uint32_t t = 0; t < kd; t++) {
        const u64 p = dst[t];
        u64* o = out + (size_t)t * n;
        memset(o, 0, sizeof(u64) * n);
        for (uint32_t i = 0; i < ks; i++) {
            u64 si = 1;
            for (uint32_t j = 0; j < ks; j++)
                if (j != i) si = mulmod(si, src[j] % p, p);
            const u64 wrap = mulmod(src[i] % p, si, p); /* src_i * S_i mod p */
            for (u64 c = 0; c < n; c++) {
                u64 yi = y[(size_t)i * n + c];
                u64 term = mulmod(yi % p, si, p);
                if (centred && yi > src[i] / 2) term = submod(term, wrap, p);
                o[c] = addmod(o[c], term, p);
            }
        }
    }
    free(y);
}

/* ---- counter-based generator (the oracle's own copy of the public recipe) ----
 * word(seed, tag, index) = M(M(seed ^ M(tag)) + index), M = the 64-bit finaliser below.
 * tag = domain | key_id << 8 | digit << 40 | limb << 48. */
static inline u64 mix64(u64 z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
static inline u64 draw(u64 seed, u64 tag, u64 index) { return mix64(mix64(seed ^ mix64(tag)) + index); }
u64 orc_draw(u64 seed, u64 tag, u64 index) { return draw(seed, tag, index); }

/* uniform modulo q: floor(word * q / 2^64) */
void orc_sample_uniform(u64 seed, u64 tag, u64 q, u64* out, u64 n) {
    for (u64 i = 0; i < n; i++) out[i] = (u64)(((u128)draw(seed, tag, i) * q) >> 64);
}
/* ternary in {-1,0,1}: floor(3*word/2^64) - 1, as int64 */
void orc_sample_ternary(u64 seed, u64 tag, int64_t* out, u64 n) {
    for (u64 i = 0; i < n; i++) out[i] = (int64_t)(((u128)draw(seed, tag, i) * 3) >> 64) - 1;
}
/* centred binomial, eta = 21: popcount(low 21 bits) - popcount(next 21 bits) */
void orc_sample_cbd(u64 seed, u64 tag, int64_t* out, u64 n) {
    const u64 m = (1ull << 21) - 1;
    for (u64 i = 0; i < n; i++) {
        u64 w = draw(seed, tag, i);
        out[i] = (int64_t)__builtin_popcountll(w & m) - (int64_t)__builtin_popcountll((w >> 21) & m);
    }
}
/* signed small integers -> residues modulo q[l], k limbs */
void orc_signed_to_rns(const int64_t* v, u64* out, const u64* q, uint32_t k, u64 n) {
    for (uint32_t l = 0; l < k; l++)
        for (u64 i = 0; i < n; i++) {
            int64_t x = v[i];
            out[l * n + i] = x >= 0 ? (u64)x % q[l] : (q[l] - ((u64)(-x) % q[l])) % q[l];
        }
}
