// Internal declarations of the sm_100a RNS-CKKS library: device arithmetic, context layout.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <map>
#include <string>
#include <vector>

#include "fesc.h"

typedef unsigned long long u64;
typedef unsigned __int128 u128;

// ---------------------------------------------------------------------------------------
// Debug build (-DFESC_DEBUG_BOUNDS -rdc=true): every kernel checks the regions its CTA (or thread) is about to touch
// against a table of known extents: the library's own allocations and the caller's buffers as registered through
// fesc_debug_bounds_register.  A region outside every extent is recorded (count, first site = file id << 16 | line,
// address, size) and the accesses to it are skipped, so that a wrong index never reaches memory; nothing traps.
// Checks sit where the outcome is the same for every thread that later meets a barrier.
// ---------------------------------------------------------------------------------------
#ifndef FESC_DBG_FILE
#define FESC_DBG_FILE 0
#endif
#ifdef FESC_DEBUG_BOUNDS
#define FESC_DBG_MAX 4096
struct DbgTable {
    uint32_t n, hits, first_site, pad;
    unsigned long long first_addr, first_bytes;
    unsigned long long lo[FESC_DBG_MAX], hi[FESC_DBG_MAX];
};
extern __device__ DbgTable g_fesc_dbg;
__device__ bool fesc_dbg_region(const void* p, size_t bytes, uint32_t site);
#define DBG_REGION(p, bytes) fesc_dbg_region((const void*)(p), (size_t)(bytes), ((uint32_t)FESC_DBG_FILE << 16) | __LINE__)
void dbg_note_alloc(const void* p, size_t bytes);
void dbg_note_free(const void* p);
#else
#define DBG_REGION(p, bytes) true
static inline void dbg_note_alloc(const void*, size_t) {}
static inline void dbg_note_free(const void*) {}
#endif

#define FESC_MAX_PRIMES 64
#define FESC_MAX_SPECIAL 8
#define FESC_MAX_ALPHA 8

// ---------------------------------------------------------------------------------------
// Per-prime constants (device copy lives in ctx->d_pc, indexed by prime index).
// ---------------------------------------------------------------------------------------
struct PrimeConst {
    u64 q;
    u64 mu;        // floor(2^64 / q)
    u64 c64;       // 2^64 mod q
    u64 c64s;      // floor(c64 * 2^64 / q)   (Shoup companion)
    u64 ninv;      // N^-1 mod q
    u64 ninvs;     // Shoup companion of ninv
    u64 ninvw;     // N^-1 * psi^-brev(1) mod q  (last inverse stage, odd output)
    u64 ninvws;
    double qd;     // q, 1/q, ninv, ninvw as doubles (exact for q < 2^50; used by the FP64 butterflies)
    double qinvd;
    double ninvd;
    double ninvwd;
};

// ---------------------------------------------------------------------------------------
// Device arithmetic.  All moduli are < 2^62, so 4q fits in 64 bits.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ u64 mulhi(u64 a, u64 b) { return __umul64hi(a, b); }

// x*w mod q in [0, 2q) for any x < 2^64, w < q, ws = floor(w*2^64/q)
__device__ __forceinline__ u64 shoup_lazy(u64 x, u64 w, u64 ws, u64 q) {
    return x * w - mulhi(x, ws) * q;
}
__device__ __forceinline__ u64 csub(u64 x, u64 q) { return x >= q ? x - q : x; }
__device__ __forceinline__ u64 shoup(u64 x, u64 w, u64 ws, u64 q) { return csub(shoup_lazy(x, w, ws, q), q); }
__device__ __forceinline__ u64 addmod(u64 a, u64 b, u64 q) { return csub(a + b, q); }
__device__ __forceinline__ u64 submod(u64 a, u64 b, u64 q) { return a >= b ? a - b : a + q - b; }

// 128-bit accumulator
struct acc128 {
    u64 lo, hi;
};
__device__ __forceinline__ void mac128(acc128& a, u64 x, u64 y) {
    u128 v = ((u128)a.hi << 64) | a.lo;
    v += (u128)x * y;
    a.lo = (u64)v;
    a.hi = (u64)(v >> 64);
}
// (hi*2^64 + lo) mod q, canonical.  hi may be any 64-bit value.
__device__ __forceinline__ u64 reduce128(u64 hi, u64 lo, const PrimeConst& pc) {
    u64 a = shoup_lazy(hi, pc.c64, pc.c64s, pc.q);     // hi*2^64 mod q, in [0,2q)
    u64 b = lo - mulhi(lo, pc.mu) * pc.q;              // lo mod q, in [0,2q)
    u64 s = a + b;                                     // < 4q < 2^64
    s = csub(s, 2 * pc.q);
    return csub(s, pc.q);
}
__device__ __forceinline__ u64 mulmod(u64 x, u64 y, const PrimeConst& pc) {
    return reduce128(mulhi(x, y), x * y, pc);
}

// ---------------------------------------------------------------------------------------
// Exact modular arithmetic on the FP64 pipe for moduli below 2^50.
// B200 issues 64 FP64 FMAs per clock per SM on a pipe of its own, while a 64x64 product costs about 26
// cycles of the 32-bit multiplier pipe per warp.  For q < 2^50 every residue is an exact double and
//     h = fl(y*w),  l = fma(y, w, -h)              (h + l = y*w exactly)
//     c = rint(h * (1/q)),  v = fma(-c, q, h) + l    (= y*w - c*q exactly, an integer below 2^53)
// is an exact signed lazy product with |v| <= (1/2 + 3 |y| 2^-53) q for |y| < 2^53, 0 <= w < q.
// Sums of such values are exact while they stay below 2^53 (8q); x - rint(x/q) q brings them back to
// |x| <= q/2.  Results equal the integer arithmetic bit for bit.
// ---------------------------------------------------------------------------------------
#define FESC_FP_LIMIT (1ull << 50)
__device__ __forceinline__ double fp_modmul(double y, double w, double q, double qinv) {
    const double h = __dmul_rn(y, w);
    const double l = __fma_rn(y, w, -h);
    const double c = rint(__dmul_rn(h, qinv));
    return __dadd_rn(__fma_rn(-c, q, h), l);
}
__device__ __forceinline__ double fp_reduce(double x, double q, double qinv) {
    return __fma_rn(-rint(__dmul_rn(x, qinv)), q, x);
}
// integer below 2^52 -> double (exact)
__device__ __forceinline__ double fp_from_u64(u64 a) {
    return __longlong_as_double((long long)(a | 0x4330000000000000ull)) - 4503599627370496.0;
}
// canonical residue -> double in [-q/2, q/2)
__device__ __forceinline__ double fp_load(u64 a, double q) {
    const double d = fp_from_u64(a);
    return d + d >= q ? d - q : d;
}
// integer-valued double below 2^53 -> canonical residue
__device__ __forceinline__ u64 fp_store(double x, double q, double qinv) {
    x = fp_reduce(x, q, qinv);
    x = x < 0.0 ? x + q : x;
    return (u64)__double_as_longlong(x + 4503599627370496.0) & 0x000FFFFFFFFFFFFFull;
}

// ---------------------------------------------------------------------------------------
// Shared-memory barriers and bulk asynchronous copies (every copy targets the issuing CTA only; no multicast).
// Every wait on a barrier is bounded: it polls a fixed number of times and reports failure instead of spinning.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// returns 0 when the phase completed, 1 when the poll budget ran out
__device__ __forceinline__ uint32_t mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    for (uint32_t it = 0; it < (1u << 20); it++) {
        if (mbar_try_wait(bar, parity)) return 0;
        if (it > 64) __nanosleep(64);
    }
    return 1;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// counter-based generator (same public recipe as the header documents)
__host__ __device__ __forceinline__ u64 mix64(u64 z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
__host__ __device__ __forceinline__ u64 make_tag(u64 domain, u64 key_id, u64 digit, u64 limb) {
    return domain | (key_id << 8) | (digit << 40) | (limb << 48);
}

// ---------------------------------------------------------------------------------------
// Row maps: which prime a row of a batched buffer uses.  Row r uses prime[r % period];
// 0xFF = skip the row.
// ---------------------------------------------------------------------------------------
struct RowMap {
    uint32_t period;
    uint8_t prime[252];
};

// ---------------------------------------------------------------------------------------
// Basis-conversion tables (device copies; built on the host in ctx.cu)
// ---------------------------------------------------------------------------------------
// One key-switch digit at one level: source limbs [first, first+n_src), Q_j = their product.
struct ModUpDigit {
    uint32_t n_src, first;
    u64 inv[FESC_MAX_ALPHA], invs[FESC_MAX_ALPHA];   // (Q_j/q_i)^-1 mod q_i and its Shoup companion
    u64 mat[FESC_MAX_ALPHA][FESC_MAX_PRIMES];        // (Q_j/q_i) mod q_t, t = prime index
    double matd[FESC_MAX_ALPHA][FESC_MAX_PRIMES];    // the same as doubles (exact for targets below 2^53)
};
// Division by P = product of the special primes p_k.
struct ModDownTab {
    u64 inv[FESC_MAX_SPECIAL], invs[FESC_MAX_SPECIAL];   // (P/p_k)^-1 mod p_k
    u64 half[FESC_MAX_SPECIAL];                          // floor(p_k / 2)
    u64 mat[FESC_MAX_SPECIAL][FESC_MAX_PRIMES];          // (P/p_k) mod q_i
    u64 mat30[FESC_MAX_SPECIAL][FESC_MAX_PRIMES];        // (P/p_k) * 2^30 mod q_i
    u64 wrap[FESC_MAX_SPECIAL + 1][FESC_MAX_PRIMES];     // cnt * P mod q_i
    u64 pinv[FESC_MAX_PRIMES], pinvs[FESC_MAX_PRIMES];   // P^-1 mod q_i
    double matd[FESC_MAX_SPECIAL][FESC_MAX_PRIMES], mat30d[FESC_MAX_SPECIAL][FESC_MAX_PRIMES];   // as doubles
    double wrapd[FESC_MAX_SPECIAL + 1][FESC_MAX_PRIMES], pinvd[FESC_MAX_PRIMES];
};
// Rescale from level l (drops limb l-1); entry index l.
struct RescaleTab {
    u64 qinv[FESC_MAX_PRIMES], qinvs[FESC_MAX_PRIMES];   // q_{l-1}^-1 mod q_i
    u64 wrap[FESC_MAX_PRIMES];                           // q_{l-1} mod q_i
    u64 half;                                            // floor(q_{l-1} / 2)
    double qinvd[FESC_MAX_PRIMES];                       // qinv as doubles (exact below 2^53)
};
struct Tables {
    ModUpDigit* d_modup;      // [(level-1) * beta_max + digit], level = 1..n_q
    ModDownTab* d_moddown;
    RescaleTab* d_rescale;    // [level], level = 2..n_q (index 0,1 unused)
    u64* d_Pmod_all;          // P mod q_t for every prime index (0 on special primes)
    uint4* d_md_frag;         // constant operand fragments of the tensor-core conversion of the division by P
                              // (bconv.cu), 512 uint4; nullptr when the shapes are not covered
};

// ---------------------------------------------------------------------------------------
// Context
// ---------------------------------------------------------------------------------------
struct EvalKey {
    u64 g;          // Galois element (0 for the relinearisation key)
    u64* d_key;     // [beta_max][2][n_q+n_p][N]
};

// Optional per-kernel-family timing with CUDA events on the launching stream.
enum { PF_NTT = 0, PF_MODUP, PF_INNER, PF_MODDOWN, PF_AUTOM, PF_BSGS, PF_RESCALE, PF_POINTWISE, PF_COUNT };
struct Profiler {
    uint32_t on = 0;               // bit f set: family f is timed
    std::vector<cudaEvent_t> ev;   // pairs (start, stop)
    std::vector<int> fam;
    size_t used = 0;
};

struct fesc_ctx {
    uint32_t log_n, N, n_q, n_p, n_primes, dnum, alpha, beta_max;
    u64 seed;
    std::vector<u64> q;           // host primes
    std::vector<PrimeConst> pc;   // host copy
    PrimeConst* d_pc;             // device [n_primes]
    ulonglong2* d_tw;             // forward twiddles [n_primes][N] (w, shoup)
    ulonglong2* d_itw;            // inverse twiddles [n_primes][N]
    double* d_twf;                // the same twiddles as doubles, rows of primes >= 2^50 unused
    double* d_itwf;
    u64* d_s;                     // secret key, EVAL, [n_primes][N]
    Tables tabs;
    std::map<uint32_t, EvalKey> keys;
    // scratch
    u64* d_scratch;
    size_t scratch_bytes;
    uint32_t fail_allocs = 0;     // test hook: this many scratch allocations report FESC_ENOMEM
    uint32_t* d_status;           // device word: non-zero after a bounded device-side wait gave up
    uint64_t counters[8];
    Profiler prof;
    std::string err;
};

static inline void prof_begin(fesc_ctx* ctx, int family, cudaStream_t st) {
    Profiler& p = ctx->prof;
    if (((p.on >> family) & 1) && p.used + 2 <= p.ev.size()) cudaEventRecord(p.ev[p.used], st);
}
static inline void prof_end(fesc_ctx* ctx, int family, cudaStream_t st, uint64_t launches = 1) {
    ctx->counters[4] += launches;
    Profiler& p = ctx->prof;
    if (((p.on >> family) & 1) && p.used + 2 <= p.ev.size()) {
        cudaEventRecord(p.ev[p.used + 1], st);
        p.fam.push_back(family);
        p.used += 2;
    }
}

#define FESC_CHECK_CUDA(ctx, call)                                                          \
    do {                                                                                    \
        cudaError_t e_ = (call);                                                            \
        if (e_ != cudaSuccess) {                                                            \
            (ctx)->err = std::string(#call) + ": " + cudaGetErrorString(e_);                \
            return FESC_ECUDA;                                                              \
        }                                                                                   \
    } while (0)

static inline int fesc_fail(fesc_ctx* ctx, int code, const std::string& msg) {
    if (ctx) ctx->err = msg;
    return code;
}

// Galois automorphism X -> X^g in evaluation (bit-reversed) order: out[t] = in[galois_src(t)]
__device__ __forceinline__ uint32_t galois_src(uint32_t t, uint32_t log_n, u64 g) {
    uint32_t u = __brev(t) >> (32 - log_n);
    uint32_t e = (uint32_t)(((2ull * u + 1) * g) & ((2ull << log_n) - 1));
    return __brev((e - 1) >> 1) >> (32 - log_n);
}

// Optional epilogue of the last pass of a forward N = 2^16 transform over rows r = bp * level + i (bp = ciphertext * 2 +
// polynomial, i = data limb, all primes below 2^50): instead of storing the transformed row u, the pass stores the last
// step of an exact division,  out[b][p][i] = (acc[bp][i] - u) * c_i  (added to what out holds when bit p of add_mask
// is set), which saves writing u, reading it back and a launch.  Division by P after a key switch: acc = the inner
// products, c_i = P^-1 mod q_i.  Rescale: acc = the input ciphertexts, c_i = q_last^-1 mod q_i, out may be the buffer
// that holds u.
struct NttFinish {
    const u64* acc = nullptr;        // ciphertext b at acc + b * acc_stride, [2][acc_rows][N]; nullptr = no epilogue
    size_t acc_stride = 0;
    u64* out = nullptr;              // ciphertext b at out + b * out_stride, [2][level][N]
    size_t out_stride = 0;
    const double* cinv = nullptr;    // device array: c_i as doubles
    uint32_t level = 0, acc_rows = 0;
    int add_mask = 0;
    // rotation: the first polynomial also receives sigma_g(c0) of the input ciphertext, read through the permutation here
    // (instead of a kernel that writes the permuted c0 to `out` first and add_mask bit 0)
    const u64* rot_src = nullptr;    // ciphertext b at rot_src + b * rot_stride, first polynomial [level][N]
    size_t rot_stride = 0;
    u64 rot_g = 0;
};

// internal launchers (ntt.cu)
// rows: number of N-word rows starting at d_data; map gives the prime per row.
// in_double (forward, N = 2^16 only): rows on primes below 2^50 hold doubles with |x| <= q/2 (bit patterns) written by a
// basis-conversion kernel instead of canonical words.
// out_double (forward, N = 2^16 only): such rows are left as doubles with |x| <= q/2 for a consumer that computes in FP64.
int ntt_launch(fesc_ctx* ctx, u64* d_data, size_t rows, const RowMap& map, bool inverse, cudaStream_t st,
               bool in_double = false, bool out_double = false, const NttFinish* finish = nullptr);
// double with |x| <= q/2 as handed to the forward transform
__device__ __forceinline__ u64 fp_handoff(double s, double q, double qinv) {
    return (u64)__double_as_longlong(fp_reduce(s, q, qinv));
}
// scratch (ctx.cu)
int ctx_scratch(fesc_ctx* ctx, size_t bytes, u64** out);
