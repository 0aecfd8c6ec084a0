// Context: parameter validation, twiddle / basis-conversion tables, seeded key generation.
#define FESC_DBG_FILE 1   // file id in the sites a debug build reports
#include "common.cuh"

#include <algorithm>

// Every device allocation of the library goes through these two, so that a debug build knows the extents.
template <typename T>
static cudaError_t dev_alloc(T** p, size_t bytes) {
    const cudaError_t e = cudaMalloc((void**)p, bytes);
    if (e == cudaSuccess) dbg_note_alloc(*p, bytes);
    return e;
}
static void dev_free(void* p) {
    if (p) dbg_note_free(p);
    cudaFree(p);
}

#ifdef FESC_DEBUG_BOUNDS
__device__ DbgTable g_fesc_dbg;
__device__ bool fesc_dbg_region(const void* p, size_t bytes, uint32_t site) {
    const unsigned long long lo = (unsigned long long)p, hi = lo + bytes;
    // the table is sorted and its ranges are disjoint: the only candidate is the last range that starts at or below lo
    uint32_t a = 0, b = g_fesc_dbg.n;
    while (a < b) {
        const uint32_t m = (a + b) >> 1;
        if (g_fesc_dbg.lo[m] <= lo) a = m + 1;
        else b = m;
    }
    if (a > 0 && hi <= g_fesc_dbg.hi[a - 1]) return true;
    if (atomicAdd(&g_fesc_dbg.hits, 1u) == 0) {
        g_fesc_dbg.first_site = site;
        g_fesc_dbg.first_addr = lo;
        g_fesc_dbg.first_bytes = bytes;
    }
    return false;
}
// Host mirror: the library's allocations and the caller's registered buffers (oldest replaced when full).
#define FESC_DBG_CALLERS 192
struct DbgHost {
    std::vector<std::pair<unsigned long long, unsigned long long>> own, caller;
};
static DbgHost& dbg_host() {
    static DbgHost h;
    return h;
}
static void dbg_upload() {
    DbgHost& h = dbg_host();
    std::vector<std::pair<unsigned long long, unsigned long long>> all(h.own);
    all.insert(all.end(), h.caller.begin(), h.caller.end());
    std::sort(all.begin(), all.end());
    static DbgTable t;      // host staging copy; the counters are left as the device has them
    uint32_t n = 0;
    for (auto& r : all) {   // overlapping ranges (a view inside a registered tensor) are joined; touching ones are not
        if (n && r.first < t.hi[n - 1]) {
            if (r.second > t.hi[n - 1]) t.hi[n - 1] = r.second;
        } else if (n < FESC_DBG_MAX) {
            t.lo[n] = r.first, t.hi[n] = r.second, n++;
        }
    }
    cudaDeviceSynchronize();
    cudaMemcpyToSymbol(g_fesc_dbg, &n, sizeof(n), offsetof(DbgTable, n));
    cudaMemcpyToSymbol(g_fesc_dbg, t.lo, sizeof(u64) * (n ? n : 1), offsetof(DbgTable, lo));
    cudaMemcpyToSymbol(g_fesc_dbg, t.hi, sizeof(u64) * (n ? n : 1), offsetof(DbgTable, hi));
}
void dbg_note_alloc(const void* p, size_t bytes) {
    dbg_host().own.push_back({(unsigned long long)p, (unsigned long long)p + bytes});
    dbg_upload();
}
void dbg_note_free(const void* p) {
    auto& v = dbg_host().own;
    for (size_t i = 0; i < v.size(); i++)
        if (v[i].first == (unsigned long long)p) {
            v.erase(v.begin() + i);
            break;
        }
    dbg_upload();
}
extern "C" int fesc_debug_bounds_register(const void* d_ptr, size_t bytes) {
    if (!d_ptr || !bytes) return FESC_EINVAL;
    DbgHost& h = dbg_host();
    const unsigned long long lo = (unsigned long long)d_ptr, hi = lo + bytes;
    // kept in order of last registration: a buffer registered again moves to the back (with its new extent), and the
    // front, the one registered longest ago, is dropped when the list is full: never a buffer of the call being set up
    bool same = false;
    for (size_t i = 0; i < h.caller.size(); i++)
        if (h.caller[i].first == lo) {
            same = h.caller[i].second == hi;
            h.caller.erase(h.caller.begin() + i);
            break;
        }
    bool dropped = false;
    if (h.caller.size() >= FESC_DBG_CALLERS) {
        h.caller.erase(h.caller.begin());
        dropped = true;
    }
    h.caller.push_back({lo, hi});
    if (!same || dropped) dbg_upload();
    return FESC_OK;
}
extern "C" int fesc_debug_bounds_clear(void) {
    dbg_host().caller.clear();
    dbg_upload();
    return FESC_OK;
}
extern "C" int fesc_debug_bounds_report(uint32_t* hits, uint32_t* first_site, uint64_t* first_addr, uint64_t* first_bytes) {
    DbgTable t;
    if (cudaDeviceSynchronize() != cudaSuccess) return FESC_ECUDA;
    if (cudaMemcpyFromSymbol(&t, g_fesc_dbg, offsetof(DbgTable, lo)) != cudaSuccess) return FESC_ECUDA;
    if (hits) *hits = t.hits;
    if (first_site) *first_site = t.first_site;
    if (first_addr) *first_addr = t.first_addr;
    if (first_bytes) *first_bytes = t.first_bytes;
    const uint32_t zero[4] = {0, 0, 0, 0};      // hits, first_site, pad: start a new record
    cudaMemcpyToSymbol(g_fesc_dbg, zero, 12, offsetof(DbgTable, hits));
    return FESC_OK;
}
#else
extern "C" int fesc_debug_bounds_register(const void*, size_t) { return FESC_EINVAL; }
extern "C" int fesc_debug_bounds_clear(void) { return FESC_EINVAL; }
extern "C" int fesc_debug_bounds_report(uint32_t*, uint32_t*, uint64_t*, uint64_t*) { return FESC_EINVAL; }
#endif

// ---------------------------------------------------------------------------------------
// host modular arithmetic (table construction only)
// ---------------------------------------------------------------------------------------
static u64 h_mul(u64 a, u64 b, u64 q) { return (u64)((u128)a * b % q); }
static u64 h_pow(u64 a, u64 e, u64 q) {
    u64 r = 1;
    a %= q;
    for (; e; e >>= 1) {
        if (e & 1) r = h_mul(r, a, q);
        a = h_mul(a, a, q);
    }
    return r;
}
static u64 h_inv(u64 a, u64 q) { return h_pow(a % q, q - 2, q); }
static u64 h_shoup(u64 w, u64 q) { return (u64)(((u128)w << 64) / q); }
static bool h_is_prime(u64 n) {
    if (n < 2) return false;
    static const u64 bases[] = {2, 3, 5, 7, 11, 13, 17, 19, 23, 29, 31, 37};
    for (u64 p : bases) {
        if (n % p == 0) return n == p;
    }
    u64 d = n - 1;
    int r = 0;
    while ((d & 1) == 0) d >>= 1, r++;
    for (u64 a : bases) {
        u64 x = h_pow(a, d, n);
        if (x == 1 || x == n - 1) continue;
        bool comp = true;
        for (int i = 1; i < r; i++) {
            x = h_mul(x, x, n);
            if (x == n - 1) {
                comp = false;
                break;
            }
        }
        if (comp) return false;
    }
    return true;
}
static uint32_t h_brev(uint32_t x, uint32_t bits) {
    uint32_t r = 0;
    for (uint32_t i = 0; i < bits; i++) r = (r << 1) | ((x >> i) & 1);
    return r;
}
// smallest primitive 2N-th root of unity
static u64 h_min_root(u64 q, uint32_t log_n) {
    const u64 N = 1ull << log_n;
    u64 root = 0;
    for (u64 g = 2; g < 4096 && !root; g++) {
        u64 c = h_pow(g, (q - 1) / (2 * N), q);
        if (h_pow(c, N, q) == q - 1) root = c;
    }
    if (!root) return 0;
    u64 sq = h_mul(root, root, q), cur = root, best = root;
    for (u64 i = 1; i < N; i++) {
        cur = h_mul(cur, sq, q);
        if (cur < best) best = cur;
    }
    return best;
}

// ---------------------------------------------------------------------------------------
// key-generation kernels
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ u64 draw(u64 seed, u64 tag, u64 idx) { return mix64(mix64(seed ^ mix64(tag)) + idx); }

// out[limb][i] uniform below q_limb, tag carries (domain, key_id, digit), limb index added here
__global__ void k_sample_uniform(u64* __restrict__ out, const PrimeConst* __restrict__ pcs, uint32_t N, u64 seed,
                                 u64 tag_base) {
    const uint32_t limb = blockIdx.y;
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    u64 w = draw(seed, tag_base | ((u64)limb << 48), i);
    if (!DBG_REGION(out + (size_t)limb * N, N * sizeof(u64))) return;
    out[(size_t)limb * N + i] = mulhi(w, pcs[limb].q);
}
// kind 0: ternary, kind 1: centred binomial (eta 21); the same small integer reduced on every limb
__global__ void k_sample_small(u64* __restrict__ out, const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t n_limbs,
                               u64 seed, u64 tag, int kind) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    u64 w = draw(seed, tag, i);
    if (!DBG_REGION(out, (size_t)n_limbs * N * sizeof(u64))) return;
    long long v;
    if (kind == 0) {
        v = (long long)mulhi(w, 3) - 1;
    } else {
        const u64 m = (1ull << 21) - 1;
        v = (long long)__popcll(w & m) - (long long)__popcll((w >> 21) & m);
    }
    for (uint32_t l = 0; l < n_limbs; l++) {
        u64 q = pcs[l].q;
        out[(size_t)l * N + i] = v >= 0 ? (u64)v : q - (u64)(-v);
    }
}
// b = -a*s + e + [limb in digit] * Pmod[limb] * sp      (all EVAL, all limbs)
__global__ void k_make_b(u64* __restrict__ b, const u64* __restrict__ a, const u64* __restrict__ s,
                         const u64* __restrict__ e, const u64* __restrict__ sp, const PrimeConst* __restrict__ pcs,
                         const u64* __restrict__ Pmod, uint32_t N, uint32_t dig_lo, uint32_t dig_hi) {
    const uint32_t limb = blockIdx.y;
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const PrimeConst pc = pcs[limb];
    const size_t o = (size_t)limb * N + i;
    if (!DBG_REGION(b + o - i, N * sizeof(u64)) || !DBG_REGION(a + o - i, N * sizeof(u64)) || !DBG_REGION(s + o - i, N * sizeof(u64)) ||
        !DBG_REGION(e + o - i, N * sizeof(u64)) || !DBG_REGION(sp + o - i, N * sizeof(u64)))
        return;
    u64 v = submod(e[o], mulmod(a[o], s[o], pc), pc.q);
    if (limb >= dig_lo && limb < dig_hi) v = addmod(v, mulmod(Pmod[limb], sp[o], pc), pc.q);
    b[o] = v;
}
__global__ void k_square(u64* __restrict__ out, const u64* __restrict__ s, const PrimeConst* __restrict__ pcs,
                         uint32_t N) {
    const uint32_t limb = blockIdx.y;
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const size_t o = (size_t)limb * N + i;
    if (!DBG_REGION(out + o - i, N * sizeof(u64)) || !DBG_REGION(s + o - i, N * sizeof(u64))) return;
    out[o] = mulmod(s[o], s[o], pcs[limb]);
}
// out[t] = in[pi_g(t)]: the Galois map in bit-reversed evaluation order
__global__ void k_autom_rows(u64* __restrict__ out, const u64* __restrict__ in, uint32_t log_n, u64 g) {
    const uint32_t N = 1u << log_n;
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= N) return;
    const size_t row = blockIdx.y;
    uint32_t u = __brev(t) >> (32 - log_n);
    uint32_t e = (uint32_t)(((2ull * u + 1) * g) & (2ull * N - 1));
    uint32_t src = __brev((e - 1) >> 1) >> (32 - log_n);
    if (src >= N || !DBG_REGION(out + row * N, N * sizeof(u64)) || !DBG_REGION(in + row * N, N * sizeof(u64))) return;
    out[row * N + t] = in[row * N + src];
}

// ---------------------------------------------------------------------------------------
int ctx_scratch(fesc_ctx* ctx, size_t bytes, u64** out) {
    if (bytes > ctx->scratch_bytes) {
        if (ctx->d_scratch) {
            FESC_CHECK_CUDA(ctx, cudaDeviceSynchronize());
            dev_free(ctx->d_scratch);
            ctx->d_scratch = nullptr;
            ctx->scratch_bytes = 0;
            ctx->counters[3] = 0;
        }
        size_t want = (bytes + (1u << 20) - 1) & ~(size_t)((1u << 20) - 1);
        const bool injected = ctx->fail_allocs > 0;       // test hook: report the failure without calling the driver
        if (injected) ctx->fail_allocs--;
        if (injected || dev_alloc(&ctx->d_scratch, want) != cudaSuccess) {
            ctx->d_scratch = nullptr;
            cudaGetLastError();
            return fesc_fail(ctx, FESC_ENOMEM, "scratch allocation of " + std::to_string(want) + " bytes failed");
        }
        ctx->scratch_bytes = want;
        ctx->counters[3] = want;
    }
    *out = ctx->d_scratch;
    return FESC_OK;
}

template <typename T>
static int upload(fesc_ctx* ctx, T** d, const std::vector<T>& h) {
    if (dev_alloc(d, h.size() * sizeof(T)) != cudaSuccess) {
        cudaGetLastError();
        return fesc_fail(ctx, FESC_ENOMEM, "table allocation failed");
    }
    FESC_CHECK_CUDA(ctx, cudaMemcpy(*d, h.data(), h.size() * sizeof(T), cudaMemcpyHostToDevice));
    return FESC_OK;
}

static RowMap all_limbs_map(const fesc_ctx* ctx) {
    RowMap m;
    m.period = ctx->n_primes;
    for (uint32_t i = 0; i < ctx->n_primes; i++) m.prime[i] = (uint8_t)i;
    return m;
}

// Basis-conversion tables, computed with 128-bit host arithmetic.
// Constant A-operand fragments of one basis conversion for mma.sync.m16n8k32 (u8): tile t of 16 target rows, byte plane a
// of the constants C(row, k, b) = M[k][row] * 256^b mod q_row, K index = 8 k + b.  Lane (g, tg) holds, for rows 16 t + g
// (x, z) and 16 t + g + 8 (y, w), the K bytes 4 tg .. 4 tg + 3 (x, y) and 16 + 4 tg .. (z, w).
template <typename F>
static void bconv_fragments(uint4* out, F C) {
    for (uint32_t t = 0; t < 2; t++)
        for (uint32_t a = 0; a < 8; a++)
            for (uint32_t lane = 0; lane < 32; lane++) {
                const uint32_t g = lane >> 2, tg = lane & 3;
                auto pack = [&](uint32_t row, uint32_t k) {
                    uint32_t w = 0;
                    for (uint32_t jj = 0; jj < 4; jj++) w |= (uint32_t)((C(row, k, 4 * (tg & 1) + jj) >> (8 * a)) & 0xff) << (8 * jj);
                    return w;
                };
                out[(t * 8 + a) * 32 + lane] = make_uint4(pack(16 * t + g, tg >> 1), pack(16 * t + g + 8, tg >> 1),
                                                          pack(16 * t + g, 2 + (tg >> 1)), pack(16 * t + g + 8, 2 + (tg >> 1)));
            }
}

static int build_tables(fesc_ctx* ctx) {
    const uint32_t nq = ctx->n_q, np = ctx->n_primes, K = ctx->n_p, alpha = ctx->alpha;
    const std::vector<u64>& q = ctx->q;
    int rc;
    // ModUp: for every level and digit
    std::vector<ModUpDigit> mu((size_t)nq * ctx->beta_max);
    memset(mu.data(), 0, mu.size() * sizeof(ModUpDigit));
    for (uint32_t level = 1; level <= nq; level++) {
        for (uint32_t j = 0; j * alpha < level; j++) {
            ModUpDigit& d = mu[(size_t)(level - 1) * ctx->beta_max + j];
            d.first = j * alpha;
            uint32_t hi = d.first + alpha < level ? d.first + alpha : level;
            d.n_src = hi - d.first;
            for (uint32_t a = 0; a < d.n_src; a++) {
                uint32_t i = d.first + a;
                // (Q_j / q_i) modulo every prime
                for (uint32_t t = 0; t < np; t++) {
                    u64 m = 1;
                    for (uint32_t b = 0; b < d.n_src; b++)
                        if (b != a) m = h_mul(m, q[d.first + b] % q[t], q[t]);
                    d.mat[a][t] = m;
                    d.matd[a][t] = (double)m;
                }
                d.inv[a] = h_inv(d.mat[a][i], q[i]);
                d.invs[a] = h_shoup(d.inv[a], q[i]);
            }
        }
    }
    if ((rc = upload(ctx, &ctx->tabs.d_modup, mu)) != FESC_OK) return rc;
    // ModDown
    std::vector<ModDownTab> mdv(1);
    ModDownTab& md = mdv[0];
    memset(&md, 0, sizeof(md));
    std::vector<u64> Pmod(np, 0);
    for (uint32_t k = 0; k < K; k++) {
        u64 pk = q[nq + k];
        u64 hat = 1;
        for (uint32_t b = 0; b < K; b++)
            if (b != k) hat = h_mul(hat, q[nq + b] % pk, pk);
        md.inv[k] = h_inv(hat, pk);
        md.invs[k] = h_shoup(md.inv[k], pk);
        md.half[k] = pk / 2;
        for (uint32_t i = 0; i < nq; i++) {
            u64 m = 1;
            for (uint32_t b = 0; b < K; b++)
                if (b != k) m = h_mul(m, q[nq + b] % q[i], q[i]);
            md.mat[k][i] = m;
            md.mat30[k][i] = h_mul(m, (1ull << 30) % q[i], q[i]);
            md.matd[k][i] = (double)md.mat[k][i];
            md.mat30d[k][i] = (double)md.mat30[k][i];
        }
    }
    for (uint32_t i = 0; i < nq; i++) {
        u64 P = 1;
        for (uint32_t b = 0; b < K; b++) P = h_mul(P, q[nq + b] % q[i], q[i]);
        Pmod[i] = P;
        md.pinv[i] = h_inv(P, q[i]);
        md.pinvs[i] = h_shoup(md.pinv[i], q[i]);
        for (uint32_t c = 0; c <= K; c++) md.wrap[c][i] = h_mul(c, P, q[i]);
        for (uint32_t c = 0; c <= K; c++) md.wrapd[c][i] = (double)md.wrap[c][i];
        md.pinvd[i] = (double)md.pinv[i];
    }
    if ((rc = upload(ctx, &ctx->tabs.d_moddown, mdv)) != FESC_OK) return rc;
    if (K <= 4) {
        std::vector<uint4> df(512);
        bconv_fragments(df.data(), [&](uint32_t row, uint32_t k, uint32_t b) -> u64 {
            if (row >= nq || k >= K) return 0;
            u64 s = 1;
            for (uint32_t e = 0; e < b; e++) s = h_mul(s, 256, q[row]);
            return h_mul(md.mat[k][row], s, q[row]);
        });
        if ((rc = upload(ctx, &ctx->tabs.d_md_frag, df)) != FESC_OK) return rc;
    }
    if ((rc = upload(ctx, &ctx->tabs.d_Pmod_all, Pmod)) != FESC_OK) return rc;
    // Rescale
    std::vector<RescaleTab> rs(nq + 1);
    memset(rs.data(), 0, rs.size() * sizeof(RescaleTab));
    for (uint32_t level = 2; level <= nq; level++) {
        u64 ql = q[level - 1];
        rs[level].half = ql / 2;
        for (uint32_t i = 0; i + 1 < level; i++) {
            rs[level].qinv[i] = h_inv(ql % q[i], q[i]);
            rs[level].qinvs[i] = h_shoup(rs[level].qinv[i], q[i]);
            rs[level].wrap[i] = ql % q[i];
            rs[level].qinvd[i] = (double)rs[level].qinv[i];
        }
    }
    return upload(ctx, &ctx->tabs.d_rescale, rs);
}
static void free_tables(fesc_ctx* ctx) {
    dev_free(ctx->tabs.d_modup);
    dev_free(ctx->tabs.d_moddown);
    dev_free(ctx->tabs.d_rescale);
    dev_free(ctx->tabs.d_Pmod_all);
    dev_free(ctx->tabs.d_md_frag);
}

// Generate the switching key from s' (EVAL on all limbs, device) to s.
static int gen_key(fesc_ctx* ctx, uint32_t key_id, const u64* d_sp, u64 g) {
    const uint32_t N = ctx->N, np = ctx->n_primes;
    const size_t limb_words = (size_t)np * N;
    u64* d_key = nullptr;
    if (dev_alloc(&d_key, (size_t)ctx->beta_max * 2 * limb_words * sizeof(u64)) != cudaSuccess) {
        cudaGetLastError();
        return fesc_fail(ctx, FESC_ENOMEM, "key allocation failed");
    }
    u64* d_e = nullptr;
    if (dev_alloc(&d_e, limb_words * sizeof(u64)) != cudaSuccess) {
        cudaGetLastError();
        dev_free(d_key);
        return fesc_fail(ctx, FESC_ENOMEM, "key allocation failed");
    }
    dim3 grid((N + 255) / 256, np);
    RowMap map = all_limbs_map(ctx);
    int rc = FESC_OK;
    for (uint32_t j = 0; j < ctx->beta_max && rc == FESC_OK; j++) {
        u64* b = d_key + (size_t)(2 * j) * limb_words;
        u64* a = b + limb_words;
        k_sample_uniform<<<grid, 256>>>(a, ctx->d_pc, N, ctx->seed, make_tag(2, key_id, j, 0));
        k_sample_small<<<(N + 255) / 256, 256>>>(d_e, ctx->d_pc, N, np, ctx->seed, make_tag(3, key_id, j, 0), 1);
        rc = ntt_launch(ctx, d_e, np, map, false, 0);
        uint32_t lo = j * ctx->alpha, hi = lo + ctx->alpha;
        if (hi > ctx->n_q) hi = ctx->n_q;
        k_make_b<<<grid, 256>>>(b, a, ctx->d_s, d_e, d_sp, ctx->d_pc, ctx->tabs.d_Pmod_all, N, lo, hi);
    }
    cudaError_t e = cudaDeviceSynchronize();
    dev_free(d_e);
    if (rc == FESC_OK && e != cudaSuccess) {
        ctx->err = std::string("key generation: ") + cudaGetErrorString(e);
        rc = FESC_ECUDA;
    }
    if (rc != FESC_OK) {
        dev_free(d_key);
        return rc;
    }
    auto it = ctx->keys.find(key_id);
    if (it != ctx->keys.end()) dev_free(it->second.d_key);
    ctx->keys[key_id] = EvalKey{g, d_key};
    return FESC_OK;
}

extern "C" int fesc_ctx_create(fesc_ctx** out, uint32_t log_n, const uint64_t* primes, uint32_t n_q, uint32_t n_p,
                               uint32_t dnum, uint64_t seed) {
    if (!out) return FESC_EINVAL;
    *out = nullptr;
    if (!primes || n_q == 0 || n_p == 0 || dnum == 0 || n_q + n_p > FESC_MAX_PRIMES || n_p > FESC_MAX_SPECIAL)
        return FESC_EINVAL;
    if (!((log_n >= 4 && log_n <= 12) || log_n == 16)) return FESC_EINVAL;
    fesc_ctx* ctx = new (std::nothrow) fesc_ctx();
    if (!ctx) return FESC_ENOMEM;
    ctx->log_n = log_n;
    ctx->N = 1u << log_n;
    ctx->n_q = n_q;
    ctx->n_p = n_p;
    ctx->n_primes = n_q + n_p;
    ctx->dnum = dnum;
    ctx->alpha = (n_q + dnum - 1) / dnum;
    ctx->beta_max = (n_q + ctx->alpha - 1) / ctx->alpha;
    ctx->seed = seed;
    ctx->d_pc = nullptr;
    ctx->d_tw = ctx->d_itw = nullptr;
    ctx->d_twf = ctx->d_itwf = nullptr;
    ctx->d_s = nullptr;
    ctx->d_scratch = nullptr;
    ctx->d_status = nullptr;
    ctx->scratch_bytes = 0;
    memset(ctx->counters, 0, sizeof(ctx->counters));
    memset(&ctx->tabs, 0, sizeof(ctx->tabs));
    const uint32_t N = ctx->N, np = ctx->n_primes;
    int rc = FESC_OK;
    auto bail = [&](int code) {
        fesc_ctx_destroy(ctx);
        return code;
    };
    if (ctx->alpha > FESC_MAX_ALPHA) return bail(FESC_EINVAL);
    // ---- validate primes, per-prime constants, twiddles ----
    std::vector<ulonglong2> tw((size_t)np * N), itw((size_t)np * N);
    std::vector<double> twf((size_t)np * N, 0.0), itwf((size_t)np * N, 0.0);
    for (uint32_t i = 0; i < np; i++) {
        u64 q = primes[i];
        if (q >= (1ull << 62) || q < 3 || (q - 1) % (2ull * N) != 0 || !h_is_prime(q)) return bail(FESC_EINVAL);
        for (uint32_t k = 0; k < i; k++)
            if (primes[k] == q) return bail(FESC_EINVAL);
        u64 psi = h_min_root(q, log_n);
        if (!psi) return bail(FESC_EINVAL);
        u64 ipsi = h_inv(psi, q);
        ctx->q.push_back(q);
        PrimeConst pc;
        pc.q = q;
        pc.mu = (u64)((((u128)1) << 64) / q);
        pc.c64 = (u64)((((u128)1) << 64) % q);
        pc.c64s = h_shoup(pc.c64, q);
        pc.ninv = h_inv(N % q, q);
        pc.ninvs = h_shoup(pc.ninv, q);
        // powers in bit-reversed order: tw[k] = psi^brev(k), itw[k] = psi^-brev(k)
        std::vector<u64> pw(N), ipw(N);
        pw[0] = ipw[0] = 1;
        for (uint32_t k = 1; k < N; k++) {
            pw[k] = h_mul(pw[k - 1], psi, q);
            ipw[k] = h_mul(ipw[k - 1], ipsi, q);
        }
        for (uint32_t k = 0; k < N; k++) {
            uint32_t r = h_brev(k, log_n);
            tw[(size_t)i * N + k] = make_ulonglong2(pw[r], h_shoup(pw[r], q));
            itw[(size_t)i * N + k] = make_ulonglong2(ipw[r], h_shoup(ipw[r], q));
            if (q < (1ull << 50)) {
                // centred representatives (|w| <= q/2) halve the rounding term of the exact FP64 product
                twf[(size_t)i * N + k] = pw[r] > q / 2 ? -(double)(q - pw[r]) : (double)pw[r];
                itwf[(size_t)i * N + k] = ipw[r] > q / 2 ? -(double)(q - ipw[r]) : (double)ipw[r];
            }
        }
        pc.ninvw = h_mul(pc.ninv, ipw[h_brev(1, log_n)], q);
        pc.ninvws = h_shoup(pc.ninvw, q);
        pc.qd = (double)q;
        pc.qinvd = 1.0 / (double)q;
        pc.ninvd = (double)pc.ninv;
        pc.ninvwd = (double)pc.ninvw;
        ctx->pc.push_back(pc);
    }
    if ((rc = upload(ctx, &ctx->d_pc, ctx->pc)) != FESC_OK) return bail(rc);
    if ((rc = upload(ctx, &ctx->d_tw, tw)) != FESC_OK) return bail(rc);
    if ((rc = upload(ctx, &ctx->d_itw, itw)) != FESC_OK) return bail(rc);
    if ((rc = upload(ctx, &ctx->d_twf, twf)) != FESC_OK) return bail(rc);
    if ((rc = upload(ctx, &ctx->d_itwf, itwf)) != FESC_OK) return bail(rc);
    if ((rc = build_tables(ctx)) != FESC_OK) return bail(rc);
    // ---- secret key and relinearisation key ----
    if (dev_alloc(&ctx->d_s, (size_t)np * N * sizeof(u64)) != cudaSuccess) return bail(FESC_ENOMEM);
    if (dev_alloc(&ctx->d_status, sizeof(uint32_t)) != cudaSuccess) return bail(FESC_ENOMEM);
    if (cudaMemset(ctx->d_status, 0, sizeof(uint32_t)) != cudaSuccess) return bail(FESC_ECUDA);
    k_sample_small<<<(N + 255) / 256, 256>>>(ctx->d_s, ctx->d_pc, N, np, seed, make_tag(1, 0, 0, 0), 0);
    if ((rc = ntt_launch(ctx, ctx->d_s, np, all_limbs_map(ctx), false, 0)) != FESC_OK) return bail(rc);
    u64* d_s2 = nullptr;
    if (dev_alloc(&d_s2, (size_t)np * N * sizeof(u64)) != cudaSuccess) return bail(FESC_ENOMEM);
    k_square<<<dim3((N + 255) / 256, np), 256>>>(d_s2, ctx->d_s, ctx->d_pc, N);
    rc = gen_key(ctx, FESC_RELIN_KEY_ID, d_s2, 0);
    dev_free(d_s2);
    if (rc != FESC_OK) return bail(rc);
    memset(ctx->counters, 0, sizeof(ctx->counters));
    *out = ctx;
    return FESC_OK;
}

extern "C" int fesc_ctx_destroy(fesc_ctx* ctx) {
    if (!ctx) return FESC_OK;
    cudaDeviceSynchronize();
    for (auto& kv : ctx->keys) dev_free(kv.second.d_key);
    for (cudaEvent_t e : ctx->prof.ev) cudaEventDestroy(e);
    dev_free(ctx->d_pc);
    dev_free(ctx->d_tw);
    dev_free(ctx->d_itw);
    dev_free(ctx->d_twf);
    dev_free(ctx->d_itwf);
    dev_free(ctx->d_s);
    dev_free(ctx->d_scratch);
    dev_free(ctx->d_status);
    free_tables(ctx);
    delete ctx;
    return FESC_OK;
}

extern "C" int fesc_ctx_trim(fesc_ctx* ctx) {
    if (!ctx) return FESC_EINVAL;
    if (ctx->d_scratch) {
        FESC_CHECK_CUDA(ctx, cudaDeviceSynchronize());
        dev_free(ctx->d_scratch);
        ctx->d_scratch = nullptr;
        ctx->scratch_bytes = 0;
        ctx->counters[3] = 0;
    }
    return FESC_OK;
}

// product of a list of primes as little-endian 64-bit words (host; exact)
static std::vector<u64> h_product(const uint64_t* p, uint32_t first, uint32_t count) {
    std::vector<u64> v(1, 1);
    for (uint32_t i = 0; i < count; i++) {
        u64 carry = 0;
        for (size_t w = 0; w < v.size(); w++) {
            const u128 t = (u128)v[w] * p[first + i] + carry;
            v[w] = (u64)t;
            carry = (u64)(t >> 64);
        }
        if (carry) v.push_back(carry);
    }
    return v;
}
static bool h_less(const std::vector<u64>& a, const std::vector<u64>& b) {
    if (a.size() != b.size()) return a.size() < b.size();
    for (size_t w = a.size(); w-- > 0;)
        if (a[w] != b[w]) return a[w] < b[w];
    return false;
}

extern "C" int fesc_params_info(uint32_t log_n, const uint64_t* primes, uint32_t n_q, uint32_t n_p, uint32_t dnum,
                                fesc_info* out) {
    if (!out || !primes || n_q == 0 || n_p == 0 || dnum == 0 || n_q + n_p > FESC_MAX_PRIMES || n_p > FESC_MAX_SPECIAL)
        return FESC_EINVAL;
    memset(out, 0, sizeof(*out));
    out->log_n = log_n;
    out->n_q = n_q;
    out->n_p = n_p;
    out->dnum = dnum;
    out->alpha = (n_q + dnum - 1) / dnum;
    out->digits = (n_q + out->alpha - 1) / out->alpha;
    const std::vector<u64> P = h_product(primes, n_q, n_p);
    for (uint32_t i = 0; i < n_p; i++) out->log2_P += log2((double)primes[n_q + i]);
    bool noisy = false;
    for (uint32_t j = 0; j < out->digits; j++) {
        const uint32_t first = j * out->alpha, cnt = n_q - first < out->alpha ? n_q - first : out->alpha;
        double lg = 0;
        for (uint32_t i = 0; i < cnt; i++) lg += log2((double)primes[first + i]);
        if (lg > out->log2_Qmax) out->log2_Qmax = lg;
        if (h_less(P, h_product(primes, first, cnt))) noisy = true;
    }
    if (noisy) out->flags |= FESC_INFO_KEYSWITCH_NOISE;
    return FESC_OK;
}

extern "C" int fesc_ctx_info(const fesc_ctx* ctx, fesc_info* out) {
    if (!ctx) return FESC_EINVAL;
    return fesc_params_info(ctx->log_n, (const uint64_t*)ctx->q.data(), ctx->n_q, ctx->n_p, ctx->dnum, out);
}

extern "C" int fesc_ctx_test_fail_allocs(fesc_ctx* ctx, uint32_t count) {
    if (!ctx) return FESC_EINVAL;
    ctx->fail_allocs = count;
    return FESC_OK;
}

extern "C" const char* fesc_last_error(const fesc_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }

extern "C" int fesc_sync(fesc_ctx* ctx, void* stream) {
    if (!ctx) return FESC_EINVAL;
    FESC_CHECK_CUDA(ctx, cudaStreamSynchronize((cudaStream_t)stream));
    FESC_CHECK_CUDA(ctx, cudaGetLastError());
    // a kernel whose bounded wait on an asynchronous copy ran out records it here
    uint32_t status = 0;
    FESC_CHECK_CUDA(ctx, cudaMemcpy(&status, ctx->d_status, sizeof(status), cudaMemcpyDeviceToHost));
    if (status) {
        cudaMemset(ctx->d_status, 0, sizeof(uint32_t));
        return fesc_fail(ctx, FESC_ETIMEOUT, "a device-side wait on an asynchronous copy gave up (code " +
                                                 std::to_string(status) + "); results of that call are invalid");
    }
#ifdef FESC_DEBUG_BOUNDS
    uint32_t hits = 0, site = 0;
    uint64_t addr = 0, bytes = 0;
    if (fesc_debug_bounds_report(&hits, &site, &addr, &bytes) != FESC_OK) return fesc_fail(ctx, FESC_ECUDA, "reading the bounds record failed");
    if (hits)
        return fesc_fail(ctx, FESC_EBOUNDS, std::to_string(hits) + " region(s) outside every known extent were skipped; first: file " +
                                                std::to_string(site >> 16) + " line " + std::to_string(site & 0xffff) + ", address " +
                                                std::to_string(addr) + ", " + std::to_string(bytes) + " bytes");
#endif
    return FESC_OK;
}

extern "C" int fesc_ctx_add_galois_key(fesc_ctx* ctx, int32_t rot, uint32_t key_id) {
    if (!ctx) return FESC_EINVAL;
    if (key_id == FESC_RELIN_KEY_ID || key_id >= (1u << 24)) return fesc_fail(ctx, FESC_EINVAL, "key id out of range");
    const u64 twoN = 2ull * ctx->N;
    u64 g;
    if (rot == FESC_CONJ) {
        g = twoN - 1;
    } else {
        const int64_t n = ctx->N / 2;
        u64 r = (u64)((((int64_t)rot % n) + n) % n);
        g = 1;
        u64 b = 5;
        for (; r; r >>= 1) {
            if (r & 1) g = g * b % twoN;
            b = b * b % twoN;
        }
    }
    u64* d_sp = nullptr;
    if (dev_alloc(&d_sp, (size_t)ctx->n_primes * ctx->N * sizeof(u64)) != cudaSuccess) {
        cudaGetLastError();
        return fesc_fail(ctx, FESC_ENOMEM, "key allocation failed");
    }
    k_autom_rows<<<dim3((ctx->N + 255) / 256, ctx->n_primes), 256>>>(d_sp, ctx->d_s, ctx->log_n, g);
    int rc = gen_key(ctx, key_id, d_sp, g);
    dev_free(d_sp);
    return rc;
}

extern "C" int fesc_ctx_export_key(fesc_ctx* ctx, uint32_t key_id, uint64_t* d_dst, void* stream) {
    if (!ctx || !d_dst) return FESC_EINVAL;
    auto it = ctx->keys.find(key_id);
    if (it == ctx->keys.end()) return fesc_fail(ctx, FESC_ENOKEY, "no key " + std::to_string(key_id));
    size_t bytes = (size_t)ctx->beta_max * 2 * ctx->n_primes * ctx->N * sizeof(u64);
    FESC_CHECK_CUDA(ctx, cudaMemcpyAsync(d_dst, it->second.d_key, bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return FESC_OK;
}
extern "C" int fesc_ctx_export_secret(fesc_ctx* ctx, uint64_t* d_dst, void* stream) {
    if (!ctx || !d_dst) return FESC_EINVAL;
    size_t bytes = (size_t)ctx->n_primes * ctx->N * sizeof(u64);
    FESC_CHECK_CUDA(ctx, cudaMemcpyAsync(d_dst, ctx->d_s, bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return FESC_OK;
}
extern "C" int fesc_profile_enable(fesc_ctx* ctx, int on, uint32_t max_records) {
    if (!ctx) return FESC_EINVAL;
    Profiler& p = ctx->prof;
    FESC_CHECK_CUDA(ctx, cudaDeviceSynchronize());
    p.used = 0;
    p.fam.clear();
    if (on) {
        while (p.ev.size() < 2 * (size_t)max_records) {
            cudaEvent_t e;
            FESC_CHECK_CUDA(ctx, cudaEventCreate(&e));
            p.ev.push_back(e);
        }
    }
    p.on = (uint32_t)on;
    return FESC_OK;
}
extern "C" int fesc_profile_read(fesc_ctx* ctx, float ms[8], uint64_t records[8]) {
    if (!ctx || !ms || !records) return FESC_EINVAL;
    Profiler& p = ctx->prof;
    FESC_CHECK_CUDA(ctx, cudaDeviceSynchronize());
    for (int i = 0; i < 8; i++) ms[i] = 0.f, records[i] = 0;
    for (size_t r = 0; r < p.fam.size(); r++) {
        float t = 0.f;
        FESC_CHECK_CUDA(ctx, cudaEventElapsedTime(&t, p.ev[2 * r], p.ev[2 * r + 1]));
        ms[p.fam[r]] += t;
        records[p.fam[r]]++;
    }
    p.used = 0;
    p.fam.clear();
    return FESC_OK;
}
extern "C" uint32_t fesc_ctx_num_digits(const fesc_ctx* ctx) { return ctx ? ctx->beta_max : 0; }
extern "C" int fesc_ctx_counters(const fesc_ctx* ctx, uint64_t out[8]) {
    if (!ctx || !out) return FESC_EINVAL;
    memcpy(out, ctx->counters, sizeof(ctx->counters));
    return FESC_OK;
}
