// Negacyclic NTT / inverse NTT over RNS limbs for sm_100a.
//
// Forward: Cooley-Tukey butterflies with psi merged into the twiddles (natural order in,
// bit-reversed evaluation order out); inverse: Gentleman-Sande with the inverse twiddles and
// N^-1 folded into the last stage.  Twiddles carry a Shoup companion so a butterfly costs one
// mul.hi.u64 and two mul.lo.u64 on the integer pipe; values stay lazily reduced ([0,4q) forward,
// [0,2q) inverse) until the last stage.
//
// N = 2^16 runs as two kernels of 8 stages each.  Every thread keeps 8 points in registers and
// does three (3+3+2) register rounds per kernel, exchanging through shared memory in between:
//   * "strided" kernel: stages whose butterfly distance is >= 256.  A CTA owns 16 adjacent
//     columns (128 B segments) of the 256 x 256 view of the limb.
//   * "contiguous" kernel: stages with distance < 256.  One WARP owns one 256-point block, so
//     the exchanges need only __syncwarp.
// N <= 2^12 runs as one shared-memory kernel per row (tests and the tiny workload).
#define FESC_DBG_FILE 2   // file id in the sites a debug build reports
#include "common.cuh"

// CTA shapes of the N = 2^16 kernels: columns per CTA of the strided kernel (x 32 sub-threads) and
// 256-point blocks (= warps) per CTA of the contiguous kernel.
#ifndef NTT_COLS
#define NTT_COLS 8
#endif
#ifndef NTT_WARPS
#define NTT_WARPS 8
#endif

// twiddle index of local stage ls (of S) for local element e with prefix pre:
//   pre * 2^ls + (e >> (S - ls))
// (pre = 1 for the strided kernel; pre = 256 + block index for the contiguous kernel).

struct Tw {
    u64 w, s;
};
__device__ __forceinline__ Tw ldtw(const ulonglong2* __restrict__ t, uint32_t i) {
    ulonglong2 v = __ldg(t + i);
    return Tw{v.x, v.y};
}

// ---- classic lazy butterflies (any q < 2^62): forward values in [0,4q), inverse in [0,2q) ----
__device__ __forceinline__ void ct_bfly(u64& x, u64& y, const Tw& t, u64 q, u64 q2) {
    u64 u = csub(x, q2);
    u64 v = shoup_lazy(y, t.w, t.s, q);
    x = u + v;
    y = u - v + q2;
}
__device__ __forceinline__ void gs_bfly(u64& x, u64& y, const Tw& t, u64 q, u64 q2) {
    u64 u = x, v = y;
    x = csub(u + v, q2);
    y = shoup_lazy(u - v + q2, t.w, t.s, q);
}

// ---- wide lazy butterflies (q < 2^54): no conditional subtraction inside the transform ----
// The high half of x*ws is taken from three of the four 32x32 partial products; it is at most 2
// below the true value, so the lazy product lands in [0,4q) instead of [0,2q).
__device__ __forceinline__ u64 mulhi_approx(u64 x, u64 y) {
    const uint32_t x0 = (uint32_t)x, x1 = (uint32_t)(x >> 32), y0 = (uint32_t)y, y1 = (uint32_t)(y >> 32);
    return (u64)x1 * y1 + __umulhi(x1, y0) + __umulhi(x0, y1);
}
__device__ __forceinline__ u64 shoup_lazy4(u64 x, u64 w, u64 ws, u64 q) { return x * w - mulhi_approx(x, ws) * q; }

// Butterfly policy.  WIDE forward: inputs below a bound Bd give outputs below Bd + 4q (16 stages from
// canonical input stay below 65q).  WIDE inverse: inputs below `off` give x below 2*off and y below 4q, so
// the offset doubles per stage (8 stages from 4q stay below 2^10 q).
template <bool WIDE>
struct Bf {
    static __device__ __forceinline__ void ct(u64& x, u64& y, const Tw& t, u64 q, u64 q2) {
        if (WIDE) {
            u64 u = x, v = shoup_lazy4(y, t.w, t.s, q);
            x = u + v;
            y = u - v + 2 * q2;
        } else {
            ct_bfly(x, y, t, q, q2);
        }
    }
    static __device__ __forceinline__ void gs(u64& x, u64& y, const Tw& t, u64 q, u64 q2, u64 off) {
        if (WIDE) {
            u64 u = x, v = y;
            x = u + v;
            y = shoup_lazy4(u - v + off, t.w, t.s, q);
        } else {
            gs_bfly(x, y, t, q, q2);
        }
    }
};

// Three forward stages on 8 registers holding elements e0 + k*d (k = 0..7); the twiddle
// indices are base indices for the first pair of each stage.
//   stage A: pairs (k,k+4), one twiddle         idxA
//   stage B: pairs (k,k+2), twiddles            idxB + (k>>2)
//   stage C: pairs (k,k+1), twiddles            idxC + (k>>1)
template <bool W>
__device__ __forceinline__ void fwd_round2(u64 (&x)[8], const ulonglong2* __restrict__ tw, uint32_t idxB,
                                           uint32_t idxC, u64 q, u64 q2) {
    Tw b0 = ldtw(tw, idxB), b1 = ldtw(tw, idxB + 1);
    Bf<W>::ct(x[0], x[2], b0, q, q2);
    Bf<W>::ct(x[1], x[3], b0, q, q2);
    Bf<W>::ct(x[4], x[6], b1, q, q2);
    Bf<W>::ct(x[5], x[7], b1, q, q2);
#pragma unroll
    for (int k = 0; k < 4; k++) {
        Tw c = ldtw(tw, idxC + k);
        Bf<W>::ct(x[2 * k], x[2 * k + 1], c, q, q2);
    }
}
template <bool W>
__device__ __forceinline__ void fwd_round3(u64 (&x)[8], const ulonglong2* __restrict__ tw, uint32_t idxA,
                                           uint32_t idxB, uint32_t idxC, u64 q, u64 q2) {
    Tw a = ldtw(tw, idxA);
#pragma unroll
    for (int k = 0; k < 4; k++) Bf<W>::ct(x[k], x[k + 4], a, q, q2);
    fwd_round2<W>(x, tw, idxB, idxC, q, q2);
}
// Inverse rounds: stages in the opposite order (C, B, then A); `off` is the wide-mode offset of the
// first stage of the round and doubles with every stage.
template <bool W>
__device__ __forceinline__ void inv_round2(u64 (&x)[8], const ulonglong2* __restrict__ tw, uint32_t idxB,
                                           uint32_t idxC, u64 q, u64 q2, u64 off) {
#pragma unroll
    for (int k = 0; k < 4; k++) {
        Tw c = ldtw(tw, idxC + k);
        Bf<W>::gs(x[2 * k], x[2 * k + 1], c, q, q2, off);
    }
    Tw b0 = ldtw(tw, idxB), b1 = ldtw(tw, idxB + 1);
    Bf<W>::gs(x[0], x[2], b0, q, q2, 2 * off);
    Bf<W>::gs(x[1], x[3], b0, q, q2, 2 * off);
    Bf<W>::gs(x[4], x[6], b1, q, q2, 2 * off);
    Bf<W>::gs(x[5], x[7], b1, q, q2, 2 * off);
}
template <bool W>
__device__ __forceinline__ void inv_round3(u64 (&x)[8], const ulonglong2* __restrict__ tw, uint32_t idxA,
                                           uint32_t idxB, uint32_t idxC, u64 q, u64 q2, u64 off) {
    inv_round2<W>(x, tw, idxB, idxC, q, q2, off);
    Tw a = ldtw(tw, idxA);
#pragma unroll
    for (int k = 0; k < 4; k++) Bf<W>::gs(x[k], x[k + 4], a, q, q2, 4 * off);
}

// ---------------------------------------------------------------------------------------
// N = 2^16, strided kernel (stages 0..7 forward / the last 8 stages inverse).
// grid = (16 column tiles, rows); block = 512 threads = 16 columns x 32 sub-threads.
// ---------------------------------------------------------------------------------------
#define N16 65536u
#define WIDE_LIMIT (1ull << 54)

template <bool INV, bool W>
__device__ __forceinline__ void strided_body(u64* __restrict__ p, u64* __restrict__ sm, const ulonglong2* __restrict__ tw,
                                             const PrimeConst& pc) {
    const u64 q = pc.q, q2 = 2 * pc.q;
    const uint32_t col = threadIdx.x & (NTT_COLS - 1), sub = threadIdx.x / NTT_COLS;
    const uint32_t h2 = sub >> 2, l2 = sub & 3;
    u64 x[8];
    if (!INV) {
        // first register round: hi = k*32 + sub, local stages 0,1,2
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = p[(size_t)(k * 32 + sub) * 256 + col];
        fwd_round3<W>(x, tw, 1, 2, 4, q, q2);
#pragma unroll
        for (int k = 0; k < 8; k++) sm[(k * 32 + sub) * NTT_COLS + col] = x[k];
        __syncthreads();
        // second register round: hi = h2*32 + k*4 + l2, local stages 3,4,5
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[(h2 * 32 + k * 4 + l2) * NTT_COLS + col];
        fwd_round3<W>(x, tw, 8 + h2, 16 + 2 * h2, 32 + 4 * h2, q, q2);
#pragma unroll
        for (int k = 0; k < 8; k++) sm[(h2 * 32 + k * 4 + l2) * NTT_COLS + col] = x[k];
        __syncthreads();
        // third register round: hi = sub*8 + k, local stages 6,7
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[(sub * 8 + k) * NTT_COLS + col];
        fwd_round2<W>(x, tw, 64 + 2 * sub, 128 + 4 * sub, q, q2);
#pragma unroll
        for (int k = 0; k < 8; k++) p[(size_t)(sub * 8 + k) * 256 + col] = x[k];  // lazily reduced
    } else {
        const u64 off = 2 * q2;   // inputs below 4q (wide) / 2q (classic) from the contiguous kernel
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = p[(size_t)(sub * 8 + k) * 256 + col];
        inv_round2<W>(x, tw, 64 + 2 * sub, 128 + 4 * sub, q, q2, off);
#pragma unroll
        for (int k = 0; k < 8; k++) sm[(sub * 8 + k) * NTT_COLS + col] = x[k];
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[(h2 * 32 + k * 4 + l2) * NTT_COLS + col];
        inv_round3<W>(x, tw, 8 + h2, 16 + 2 * h2, 32 + 4 * h2, q, q2, 4 * off);
#pragma unroll
        for (int k = 0; k < 8; k++) sm[(h2 * 32 + k * 4 + l2) * NTT_COLS + col] = x[k];
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[(k * 32 + sub) * NTT_COLS + col];
        // stages 2,1 then the last stage with N^-1 folded in (exact products, canonical output)
        {
#pragma unroll
            for (int k = 0; k < 4; k++) {
                Tw c = ldtw(tw, 4 + k);
                Bf<W>::gs(x[2 * k], x[2 * k + 1], c, q, q2, 32 * off);
            }
            Tw b0 = ldtw(tw, 2), b1 = ldtw(tw, 3);
            Bf<W>::gs(x[0], x[2], b0, q, q2, 64 * off);
            Bf<W>::gs(x[1], x[3], b0, q, q2, 64 * off);
            Bf<W>::gs(x[4], x[6], b1, q, q2, 64 * off);
            Bf<W>::gs(x[5], x[7], b1, q, q2, 64 * off);
            const u64 last = W ? 128 * off : q2;
#pragma unroll
            for (int k = 0; k < 4; k++) {
                u64 u = x[k], v = x[k + 4];
                x[k] = shoup(u + v, pc.ninv, pc.ninvs, q);
                x[k + 4] = shoup(u - v + last, pc.ninvw, pc.ninvws, q);
            }
        }
#pragma unroll
        for (int k = 0; k < 8; k++) p[(size_t)(k * 32 + sub) * 256 + col] = x[k];
    }
}

__device__ __forceinline__ uint32_t pad8(uint32_t e) { return e + (e >> 3); }

// ---------------------------------------------------------------------------------------
// FP64 butterflies for primes below 2^50.
// B200 issues 64 FP64 FMAs per clock per SM on a pipe of its own, while a 64-bit modular product on
// the integer side costs about 40 cycles of the 32-bit multiplier pipe per warp.  For q < 2^50 every
// residue and every lazily reduced value below 2^53 is an exact double, and
//     h = fl(y*w),  l = fma(y, w, -h)           (h + l = y*w exactly)
//     c = rint(h * (1/q)),  v = fma(-c, q, h) + l (= y*w - c*q exactly, an integer below 2^53)
// is an exact signed lazy product: |v| <= (1/2 + 3|y w| 2^-53 / q) q, i.e. (1/2 + 1.5 |y| 2^-53) q with the
// twiddles stored as centred doubles (|w| <= q/2).  Sums and differences of such values are exact while they
// stay below 2^53 = 8q.  Forward (Cooley-Tukey: x +- v, bound B -> 1.1875 B + q/2 per stage): from q/2 the bound
// after 1..7 stages is 1.10, 1.80, 2.64, 3.63, 4.81, 6.21, 7.88 q, and from a canonical input (below q) three
// stages reach 3.47q; so the strided kernel folds back once after its first round and once at the end, the
// contiguous kernel once after its first round.  Inverse (Gentleman-Sande: x + v doubles the bound): three
// stages from q/2 reach 4q, so every round ends with a fold-back x - rint(x/q) q to |x| <= q/2.
// The result equals the integer transform bit for bit.
// The two kernels of one transform hand the data over as doubles in the caller's buffer.
// ---------------------------------------------------------------------------------------
#define FP_LIMIT FESC_FP_LIMIT
__device__ __forceinline__ double ldf(const double* __restrict__ t, uint32_t i) { return __ldg(t + i); }
__device__ __forceinline__ void fp_ct(double& x, double& y, double w, double q, double qinv) {
    const double v = fp_modmul(y, w, q, qinv), u = x;
    x = u + v;
    y = u - v;
}
__device__ __forceinline__ void fp_gs(double& x, double& y, double w, double q, double qinv) {
    const double u = x, v = y;
    x = u + v;
    y = fp_modmul(u - v, w, q, qinv);
}
// idxB is even and idxC a multiple of 4 at every call site: 16-byte loads
__device__ __forceinline__ double2 ldf2(const double* __restrict__ t, uint32_t i) {
    return __ldg(reinterpret_cast<const double2*>(t + i));
}
__device__ __forceinline__ void fp_fwd_round2(double (&x)[8], const double* __restrict__ tw, uint32_t idxB, uint32_t idxC,
                                              double q, double qinv) {
    const double2 b = ldf2(tw, idxB), c0 = ldf2(tw, idxC), c1 = ldf2(tw, idxC + 2);
    fp_ct(x[0], x[2], b.x, q, qinv);
    fp_ct(x[1], x[3], b.x, q, qinv);
    fp_ct(x[4], x[6], b.y, q, qinv);
    fp_ct(x[5], x[7], b.y, q, qinv);
    fp_ct(x[0], x[1], c0.x, q, qinv);
    fp_ct(x[2], x[3], c0.y, q, qinv);
    fp_ct(x[4], x[5], c1.x, q, qinv);
    fp_ct(x[6], x[7], c1.y, q, qinv);
}
__device__ __forceinline__ void fp_fwd_round3(double (&x)[8], const double* __restrict__ tw, uint32_t idxA, uint32_t idxB,
                                              uint32_t idxC, double q, double qinv) {
    const double a = ldf(tw, idxA);
#pragma unroll
    for (int k = 0; k < 4; k++) fp_ct(x[k], x[k + 4], a, q, qinv);
    fp_fwd_round2(x, tw, idxB, idxC, q, qinv);
}
__device__ __forceinline__ void fp_inv_round2(double (&x)[8], const double* __restrict__ tw, uint32_t idxB, uint32_t idxC,
                                              double q, double qinv) {
    const double2 b = ldf2(tw, idxB), c0 = ldf2(tw, idxC), c1 = ldf2(tw, idxC + 2);
    fp_gs(x[0], x[1], c0.x, q, qinv);
    fp_gs(x[2], x[3], c0.y, q, qinv);
    fp_gs(x[4], x[5], c1.x, q, qinv);
    fp_gs(x[6], x[7], c1.y, q, qinv);
    fp_gs(x[0], x[2], b.x, q, qinv);
    fp_gs(x[1], x[3], b.x, q, qinv);
    fp_gs(x[4], x[6], b.y, q, qinv);
    fp_gs(x[5], x[7], b.y, q, qinv);
}
__device__ __forceinline__ void fp_inv_round3(double (&x)[8], const double* __restrict__ tw, uint32_t idxA, uint32_t idxB,
                                              uint32_t idxC, double q, double qinv) {
    fp_inv_round2(x, tw, idxB, idxC, q, qinv);
    const double a = ldf(tw, idxA);
#pragma unroll
    for (int k = 0; k < 4; k++) fp_gs(x[k], x[k + 4], a, q, qinv);
}
__device__ __forceinline__ void fp_reduce8(double (&x)[8], double q, double qinv) {
#pragma unroll
    for (int k = 0; k < 8; k++) x[k] = fp_reduce(x[k], q, qinv);
}

template <bool INV>
__device__ __forceinline__ void strided_body_fp(u64* __restrict__ p, double* __restrict__ sm, const double* __restrict__ tw,
                                                const PrimeConst& pc, int in_double) {
    const double q = pc.qd, qinv = pc.qinvd;
    const uint32_t col = threadIdx.x & (NTT_COLS - 1), sub = threadIdx.x / NTT_COLS;
    const uint32_t h2 = sub >> 2, l2 = sub & 3;
    double x[8];
    if (!INV) {
#pragma unroll
        for (int k = 0; k < 8; k++) {   // canonical words (below q), or doubles with |x| <= q/2 from a conversion kernel
            const u64 v = p[(size_t)(k * 32 + sub) * 256 + col];
            x[k] = in_double ? __longlong_as_double((long long)v) : fp_from_u64(v);
        }
        fp_fwd_round3(x, tw, 1, 2, 4, q, qinv);                                                  // below 3.47q
        fp_reduce8(x, q, qinv);
#pragma unroll
        for (int k = 0; k < 8; k++) sm[(k * 32 + sub) * NTT_COLS + col] = x[k];
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[(h2 * 32 + k * 4 + l2) * NTT_COLS + col];
        fp_fwd_round3(x, tw, 8 + h2, 16 + 2 * h2, 32 + 4 * h2, q, qinv);                        // below 2.64q, 4.81q next
#pragma unroll
        for (int k = 0; k < 8; k++) sm[(h2 * 32 + k * 4 + l2) * NTT_COLS + col] = x[k];
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[(sub * 8 + k) * NTT_COLS + col];
        fp_fwd_round2(x, tw, 64 + 2 * sub, 128 + 4 * sub, q, qinv);
        fp_reduce8(x, q, qinv);
        // handed to the contiguous kernel as doubles, |x| <= q/2
#pragma unroll
        for (int k = 0; k < 8; k++) p[(size_t)(sub * 8 + k) * 256 + col] = (u64)__double_as_longlong(x[k]);
    } else {
        // doubles with |x| <= q/2 from the contiguous kernel
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = __longlong_as_double((long long)p[(size_t)(sub * 8 + k) * 256 + col]);
        fp_inv_round2(x, tw, 64 + 2 * sub, 128 + 4 * sub, q, qinv);
        fp_reduce8(x, q, qinv);
#pragma unroll
        for (int k = 0; k < 8; k++) sm[(sub * 8 + k) * NTT_COLS + col] = x[k];
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[(h2 * 32 + k * 4 + l2) * NTT_COLS + col];
        fp_inv_round3(x, tw, 8 + h2, 16 + 2 * h2, 32 + 4 * h2, q, qinv);
        fp_reduce8(x, q, qinv);
#pragma unroll
        for (int k = 0; k < 8; k++) sm[(h2 * 32 + k * 4 + l2) * NTT_COLS + col] = x[k];
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[(k * 32 + sub) * NTT_COLS + col];
        // stages 2, 1, then the last stage with N^-1 folded in
#pragma unroll
        for (int k = 0; k < 4; k++) fp_gs(x[2 * k], x[2 * k + 1], ldf(tw, 4 + k), q, qinv);
        {
            const double b0 = ldf(tw, 2), b1 = ldf(tw, 3);
            fp_gs(x[0], x[2], b0, q, qinv);
            fp_gs(x[1], x[3], b0, q, qinv);
            fp_gs(x[4], x[6], b1, q, qinv);
            fp_gs(x[5], x[7], b1, q, qinv);
        }
#pragma unroll
        for (int k = 0; k < 4; k++) {
            const double u = x[k], v = x[k + 4];
            x[k] = fp_modmul(u + v, pc.ninvd, q, qinv);
            x[k + 4] = fp_modmul(u - v, pc.ninvwd, q, qinv);
        }
#pragma unroll
        for (int k = 0; k < 8; k++) p[(size_t)(k * 32 + sub) * 256 + col] = fp_store(x[k], q, qinv);
    }
}

template <bool INV>
__device__ __forceinline__ void contig_body_fp(u64* __restrict__ p, double* __restrict__ sm, const double* __restrict__ tw,
                                               const PrimeConst& pc, uint32_t pre, int out_double,
                                               const u64* __restrict__ fin_acc = nullptr, u64* __restrict__ fin_out = nullptr,
                                               double fin_pinv = 0.0, int fin_add = 0, const u64* __restrict__ fin_rot = nullptr,
                                               u64 fin_g = 0, uint32_t fin_t0 = 0) {
    const double q = pc.qd, qinv = pc.qinvd;
    const uint32_t sub = threadIdx.x & 31;
    const uint32_t h2 = sub >> 2, l2 = sub & 3;
    double x[8];
    if (!INV) {
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = __longlong_as_double((long long)p[k * 32 + sub]);   // |x| <= q/2
        fp_fwd_round3(x, tw, pre, 2 * pre, 4 * pre, q, qinv);
        fp_reduce8(x, q, qinv);
#pragma unroll
        for (int k = 0; k < 8; k++) sm[pad8(k * 32 + sub)] = x[k];
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[pad8(h2 * 32 + k * 4 + l2)];
        fp_fwd_round3(x, tw, 8 * pre + h2, 16 * pre + 2 * h2, 32 * pre + 4 * h2, q, qinv);   // below 2.64q, 4.81q next
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; k++) sm[pad8(h2 * 32 + k * 4 + l2)] = x[k];
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[pad8(sub * 8 + k)];
        fp_fwd_round2(x, tw, 64 * pre + 2 * sub, 128 * pre + 4 * sub, q, qinv);
        if (fin_acc) {
            // last step of the division by P on the fly: (acc - u) * P^-1 (+ what the output holds); |acc - u| stays
            // below 6q, the lazy product below 3q, so every sum is exact
            const ulonglong2* a = reinterpret_cast<const ulonglong2*>(fin_acc + sub * 8);
            ulonglong2* o = reinterpret_cast<ulonglong2*>(fin_out + sub * 8);
#pragma unroll
            for (int k = 0; k < 4; k++) {
                const ulonglong2 av = a[k];
                double s0 = fp_modmul(fp_load(av.x, q) - x[2 * k], fin_pinv, q, qinv);
                double s1 = fp_modmul(fp_load(av.y, q) - x[2 * k + 1], fin_pinv, q, qinv);
                if (fin_rot) {        // + sigma_g(c0): the row of the input read through the permutation
                    s0 += fp_load(fin_rot[galois_src(fin_t0 + sub * 8 + 2 * k, 16, fin_g)], q);
                    s1 += fp_load(fin_rot[galois_src(fin_t0 + sub * 8 + 2 * k + 1, 16, fin_g)], q);
                }
                if (fin_add) {
                    const ulonglong2 ov = o[k];
                    s0 += fp_load(ov.x, q);
                    s1 += fp_load(ov.y, q);
                }
                o[k] = make_ulonglong2(fp_store(s0, q, qinv), fp_store(s1, q, qinv));
            }
            return;
        }
        ulonglong2* o = reinterpret_cast<ulonglong2*>(p + sub * 8);
#pragma unroll
        for (int k = 0; k < 4; k++)   // canonical words, or doubles with |x| <= q/2 for a consumer that computes in FP64
            o[k] = out_double ? make_ulonglong2(fp_handoff(x[2 * k], q, qinv), fp_handoff(x[2 * k + 1], q, qinv))
                              : make_ulonglong2(fp_store(x[2 * k], q, qinv), fp_store(x[2 * k + 1], q, qinv));
    } else {
        const ulonglong2* in = reinterpret_cast<const ulonglong2*>(p + sub * 8);
#pragma unroll
        for (int k = 0; k < 4; k++) {
            ulonglong2 v = in[k];
            x[2 * k] = fp_load(v.x, q);
            x[2 * k + 1] = fp_load(v.y, q);
        }
        fp_inv_round2(x, tw, 64 * pre + 2 * sub, 128 * pre + 4 * sub, q, qinv);
        fp_reduce8(x, q, qinv);
#pragma unroll
        for (int k = 0; k < 8; k++) sm[pad8(sub * 8 + k)] = x[k];
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[pad8(h2 * 32 + k * 4 + l2)];
        fp_inv_round3(x, tw, 8 * pre + h2, 16 * pre + 2 * h2, 32 * pre + 4 * h2, q, qinv);
        fp_reduce8(x, q, qinv);
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; k++) sm[pad8(h2 * 32 + k * 4 + l2)] = x[k];
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[pad8(k * 32 + sub)];
        fp_inv_round3(x, tw, pre, 2 * pre, 4 * pre, q, qinv);
        fp_reduce8(x, q, qinv);
#pragma unroll
        for (int k = 0; k < 8; k++) p[k * 32 + sub] = (u64)__double_as_longlong(x[k]);   // doubles, |x| <= q/2
    }
}

template <bool INV>
__global__ void __launch_bounds__(NTT_COLS * 32) ntt16_strided(u64* __restrict__ data, const ulonglong2* __restrict__ tw_all,
                                                     const double* __restrict__ twf_all,
                                                     const PrimeConst* __restrict__ pcs, RowMap map,
                                                     uint32_t row_base, int in_double) {
    const uint32_t row = blockIdx.y;
    const uint32_t pi = map.prime[(row_base + row) % map.period];
    if (pi == 0xFF) return;
    __shared__ u64 sm[256 * NTT_COLS];
    const PrimeConst pc = pcs[pi];
    const ulonglong2* tw = tw_all + (size_t)pi * N16;
    u64* p = data + (size_t)row * N16 + blockIdx.x * NTT_COLS;
    if (!DBG_REGION(data + (size_t)row * N16, N16 * sizeof(u64))) return;   // the CTA's columns span the whole row
    if (pc.q < FP_LIMIT)
        strided_body_fp<INV>(p, reinterpret_cast<double*>(sm), twf_all + (size_t)pi * N16, pc, in_double);
    else if (pc.q < WIDE_LIMIT)
        strided_body<INV, true>(p, sm, tw, pc);
    else
        strided_body<INV, false>(p, sm, tw, pc);
}

// ---------------------------------------------------------------------------------------
// N = 2^16, contiguous kernel (stages 8..15 forward / the first 8 stages inverse).
// grid = (16 tiles of 4096 points, rows); block = 512 threads = 16 warps, one 256-point block each.
// Shared exchange buffer per warp: 256 points padded to e + (e >> 3) to avoid bank conflicts.
// ---------------------------------------------------------------------------------------

template <bool INV, bool W>
__device__ __forceinline__ void contig_body(u64* __restrict__ p, u64* __restrict__ sm, const ulonglong2* __restrict__ tw,
                                            const PrimeConst& pc, uint32_t pre) {
    const u64 q = pc.q, q2 = 2 * pc.q;
    const uint32_t sub = threadIdx.x & 31;
    const uint32_t h2 = sub >> 2, l2 = sub & 3;
    u64 x[8];
    if (!INV) {
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = p[k * 32 + sub];   // lazily reduced by the strided kernel
        fwd_round3<W>(x, tw, pre, 2 * pre, 4 * pre, q, q2);
#pragma unroll
        for (int k = 0; k < 8; k++) sm[pad8(k * 32 + sub)] = x[k];
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[pad8(h2 * 32 + k * 4 + l2)];
        fwd_round3<W>(x, tw, 8 * pre + h2, 16 * pre + 2 * h2, 32 * pre + 4 * h2, q, q2);
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; k++) sm[pad8(h2 * 32 + k * 4 + l2)] = x[k];
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[pad8(sub * 8 + k)];
        fwd_round2<W>(x, tw, 64 * pre + 2 * sub, 128 * pre + 4 * sub, q, q2);
#pragma unroll
        for (int k = 0; k < 8; k++) {
            if (W) x[k] = x[k] - mulhi_approx(x[k], pc.mu) * q;   // below 65q -> below 4q
            x[k] = csub(csub(x[k], q2), q);
        }
        ulonglong2* o = reinterpret_cast<ulonglong2*>(p + sub * 8);
#pragma unroll
        for (int k = 0; k < 4; k++) o[k] = make_ulonglong2(x[2 * k], x[2 * k + 1]);
    } else {
        const u64 off = 2 * q2;   // canonical input is below 4q
        const ulonglong2* in = reinterpret_cast<const ulonglong2*>(p + sub * 8);
#pragma unroll
        for (int k = 0; k < 4; k++) {
            ulonglong2 v = in[k];
            x[2 * k] = v.x;
            x[2 * k + 1] = v.y;
        }
        inv_round2<W>(x, tw, 64 * pre + 2 * sub, 128 * pre + 4 * sub, q, q2, off);
#pragma unroll
        for (int k = 0; k < 8; k++) sm[pad8(sub * 8 + k)] = x[k];
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[pad8(h2 * 32 + k * 4 + l2)];
        inv_round3<W>(x, tw, 8 * pre + h2, 16 * pre + 2 * h2, 32 * pre + 4 * h2, q, q2, 4 * off);
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; k++) sm[pad8(h2 * 32 + k * 4 + l2)] = x[k];
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; k++) x[k] = sm[pad8(k * 32 + sub)];
        inv_round3<W>(x, tw, pre, 2 * pre, 4 * pre, q, q2, 32 * off);
#pragma unroll
        for (int k = 0; k < 8; k++) {
            if (W) x[k] = x[k] - mulhi_approx(x[k], pc.mu) * q;   // below 2^10 q -> below 4q
            p[k * 32 + sub] = x[k];                               // finished by the strided kernel
        }
    }
}

template <bool INV>
__global__ void __launch_bounds__(NTT_WARPS * 32) ntt16_contig(u64* __restrict__ data, const ulonglong2* __restrict__ tw_all,
                                                    const double* __restrict__ twf_all,
                                                    const PrimeConst* __restrict__ pcs, RowMap map,
                                                    uint32_t row_base, int out_double, NttFinish fin, uint32_t row_first) {
    const uint32_t row = blockIdx.y;
    const uint32_t pi = map.prime[(row_base + row) % map.period];
    if (pi == 0xFF) return;
    __shared__ u64 sm_all[NTT_WARPS * 288];
    const PrimeConst pc = pcs[pi];
    const ulonglong2* tw = tw_all + (size_t)pi * N16;
    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t blk = blockIdx.x * NTT_WARPS + warp;   // 256-point block index within the limb
    u64* p = data + (size_t)row * N16 + (size_t)blk * 256;
    u64* sm = sm_all + warp * 288;
    if (!DBG_REGION(p, 256 * sizeof(u64))) return;      // one warp per 256-point block, warp barriers only
    if (pc.q < FP_LIMIT) {
        if (!INV && fin.acc) {      // rows of this launch: r = bp * level + i
            const uint32_t r = row_first + row, bp = r / fin.level, i = r - bp * fin.level;
            if (!DBG_REGION(fin.acc + (size_t)(bp >> 1) * fin.acc_stride + ((size_t)(bp & 1) * fin.acc_rows + i) * N16 + (size_t)blk * 256, 256 * sizeof(u64)) ||
                !DBG_REGION(fin.out + (size_t)(bp >> 1) * fin.out_stride + ((size_t)(bp & 1) * fin.level + i) * N16 + (size_t)blk * 256,
                            256 * sizeof(u64)) ||
                (fin.rot_src && !DBG_REGION(fin.rot_src + (size_t)(bp >> 1) * fin.rot_stride + (size_t)i * N16, N16 * sizeof(u64))))
                return;
            contig_body_fp<INV>(p, reinterpret_cast<double*>(sm), twf_all + (size_t)pi * N16, pc, 256 + blk, out_double,
                                fin.acc + (size_t)(bp >> 1) * fin.acc_stride + ((size_t)(bp & 1) * fin.acc_rows + i) * N16 + (size_t)blk * 256,
                                fin.out + (size_t)(bp >> 1) * fin.out_stride + ((size_t)(bp & 1) * fin.level + i) * N16 + (size_t)blk * 256,
                                fin.cinv[i], (fin.add_mask >> (bp & 1)) & 1,
                                (fin.rot_src && !(bp & 1)) ? fin.rot_src + (size_t)(bp >> 1) * fin.rot_stride + (size_t)i * N16 : nullptr,
                                fin.rot_g, blk * 256);
        } else {
            contig_body_fp<INV>(p, reinterpret_cast<double*>(sm), twf_all + (size_t)pi * N16, pc, 256 + blk, out_double);
        }
    } else if (pc.q < WIDE_LIMIT)
        contig_body<INV, true>(p, sm, tw, pc, 256 + blk);
    else
        contig_body<INV, false>(p, sm, tw, pc, 256 + blk);
}

// ---------------------------------------------------------------------------------------
// N <= 2^12: one CTA per row, radix-2 stages in shared memory.
// ---------------------------------------------------------------------------------------
template <bool INV>
__global__ void __launch_bounds__(256) ntt_small(u64* __restrict__ data, const ulonglong2* __restrict__ tw_all,
                                                 const PrimeConst* __restrict__ pcs, RowMap map, uint32_t log_n) {
    const uint32_t row = blockIdx.x;
    const uint32_t pi = map.prime[row % map.period];
    if (pi == 0xFF) return;
    extern __shared__ u64 smx[];
    const uint32_t N = 1u << log_n;
    const PrimeConst pc = pcs[pi];
    const u64 q = pc.q, q2 = 2 * pc.q;
    const ulonglong2* tw = tw_all + (size_t)pi * N;
    u64* p = data + (size_t)row * N;
    if (!DBG_REGION(p, N * sizeof(u64)) || !DBG_REGION(tw, N * sizeof(ulonglong2))) return;
    for (uint32_t i = threadIdx.x; i < N; i += blockDim.x) smx[i] = p[i];
    __syncthreads();
    if (!INV) {
        for (uint32_t s = 0; s < log_n; s++) {
            const uint32_t t = N >> (s + 1);
            for (uint32_t b = threadIdx.x; b < N / 2; b += blockDim.x) {
                uint32_t i = b / t, k = b % t;
                uint32_t j = i * 2 * t + k;
                Tw w = ldtw(tw, (1u << s) + i);
                u64 x = smx[j], y = smx[j + t];
                ct_bfly(x, y, w, q, q2);
                smx[j] = x;
                smx[j + t] = y;
            }
            __syncthreads();
        }
        for (uint32_t i = threadIdx.x; i < N; i += blockDim.x) p[i] = csub(csub(smx[i], q2), q);
    } else {
        for (int s = (int)log_n - 1; s >= 1; s--) {
            const uint32_t t = N >> (s + 1);
            for (uint32_t b = threadIdx.x; b < N / 2; b += blockDim.x) {
                uint32_t i = b / t, k = b % t;
                uint32_t j = i * 2 * t + k;
                Tw w = ldtw(tw, (1u << s) + i);
                u64 x = smx[j], y = smx[j + t];
                gs_bfly(x, y, w, q, q2);
                smx[j] = x;
                smx[j + t] = y;
            }
            __syncthreads();
        }
        const uint32_t t = N / 2;
        for (uint32_t b = threadIdx.x; b < N / 2; b += blockDim.x) {
            u64 u = smx[b], v = smx[b + t];
            p[b] = shoup(u + v, pc.ninv, pc.ninvs, q);
            p[b + t] = shoup(u - v + q2, pc.ninvw, pc.ninvws, q);
        }
    }
}

int ntt_launch(fesc_ctx* ctx, u64* d_data, size_t rows, const RowMap& map, bool inverse, cudaStream_t st, bool in_double,
               bool out_double, const NttFinish* finish) {
    const NttFinish fin = finish ? *finish : NttFinish();
    if (fin.acc && (inverse || ctx->log_n != 16)) return fesc_fail(ctx, FESC_EINVAL, "ntt: the fused epilogue belongs to a forward N = 2^16 transform");
    if (rows == 0) return FESC_OK;
    if (rows > 0x7fffffffu) return fesc_fail(ctx, FESC_EINVAL, "ntt: too many rows");
    const ulonglong2* tw = inverse ? ctx->d_itw : ctx->d_tw;
    const double* twf = inverse ? ctx->d_itwf : ctx->d_twf;
    size_t live = 0;
    for (uint32_t i = 0; i < map.period; i++) live += map.prime[i] != 0xFF;
    ctx->counters[0] += rows / map.period * live;
    prof_begin(ctx, PF_NTT, st);
    uint64_t launches = 0;
    if (ctx->log_n == 16) {
        // gridDim.y is limited to 65535 rows per launch.  (Splitting into L2-sized chunks was measured:
        // slower, the extra launch tails cost more than the L2 hits save.)
        const size_t chunk_rows = 65535;
        for (size_t r0 = 0; r0 < rows; r0 += chunk_rows) {
            const size_t chunk = rows - r0 < chunk_rows ? rows - r0 : chunk_rows;
            const uint32_t rb = (uint32_t)(r0 % map.period);
            dim3 gs(256 / NTT_COLS, (unsigned)chunk), gc(256 / NTT_WARPS, (unsigned)chunk);
            u64* base = d_data + r0 * (size_t)N16;
            if (!inverse) {
                ntt16_strided<false><<<gs, NTT_COLS * 32, 0, st>>>(base, tw, twf, ctx->d_pc, map, rb, in_double ? 1 : 0);
                ntt16_contig<false><<<gc, NTT_WARPS * 32, 0, st>>>(base, tw, twf, ctx->d_pc, map, rb, out_double ? 1 : 0, fin, (uint32_t)r0);
            } else {
                ntt16_contig<true><<<gc, NTT_WARPS * 32, 0, st>>>(base, tw, twf, ctx->d_pc, map, rb, 0, NttFinish(), 0u);
                ntt16_strided<true><<<gs, NTT_COLS * 32, 0, st>>>(base, tw, twf, ctx->d_pc, map, rb, 0);
            }
            launches += 2;
        }
    } else {
        size_t smem = sizeof(u64) << ctx->log_n;
        if (!inverse)
            ntt_small<false><<<(unsigned)rows, 256, smem, st>>>(d_data, tw, ctx->d_pc, map, ctx->log_n);
        else
            ntt_small<true><<<(unsigned)rows, 256, smem, st>>>(d_data, tw, ctx->d_pc, map, ctx->log_n);
        launches = 1;
    }
    prof_end(ctx, PF_NTT, st, launches);
    FESC_CHECK_CUDA(ctx, cudaGetLastError());
    return FESC_OK;
}
