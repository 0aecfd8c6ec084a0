// Factorized scan-contract on packed ciphertexts:
//   h_k = br(a_k) (.) h_{k-1} + x_k (x) B_k,  h_0 = 0,   m_k = Sigma_{d_s}(h_k (.) br(C_k))
// evaluated as: per token block, broadcast of the compact factors to the state packing (rotations,
// masks, rotate-and-add fills; optionally for groups of tokens at once), leaves (p, s) = (br a, br x (.) br B),
// a prefix network (Brent-Kung, Kogge-Stone or Sklansky) of affine
// compositions (p_R p_L, p_R s_L + s_R), serialized block carries, carry injection, contraction with
// br(C), a complex-paired rotate-add reduction over the state axis with one conjugation per chunk
// pair, output mask and placement.  The host code below only sequences batched kernels (rotations
// share a key per batch); every arithmetic step runs in the kernels of ops.cu / ntt.cu and the
// pointwise kernels here.  Levels follow a fixed schedule (see fesc.h).
#include <math.h>

#include <map>

#define FESC_DBG_FILE 6   // file id in the sites a debug build reports
#include "ops.cuh"

// ---------------------------------------------------------------------------------------
// pointwise kernels on batches of compact ciphertexts [2][level][N]
// ---------------------------------------------------------------------------------------
// out = a + b (sub = 0) or a - b (sub = 1); b_stride may be 0
__global__ void __launch_bounds__(256) k_ct_addsub(const u64* __restrict__ a, size_t a_stride, const u64* __restrict__ b,
                                                   size_t b_stride, u64* __restrict__ out, size_t out_stride,
                                                   const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level,
                                                   int sub) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t pl = blockIdx.y, bi = blockIdx.z;   // pl = poly*level + limb
    if (c >= N) return;
    const u64 q = pcs[pl % level].q;
    const size_t o = (size_t)pl * N + c;
    if (!DBG_REGION(a + bi * a_stride + o - c, N * sizeof(u64)) || !DBG_REGION(b + bi * b_stride + o - c, N * sizeof(u64)) ||
        !DBG_REGION(out + bi * out_stride + o - c, N * sizeof(u64)))
        return;
    const u64 x = a[bi * a_stride + o], y = b[bi * b_stride + o];
    out[bi * out_stride + o] = sub ? submod(x, y, q) : addmod(x, y, q);
}
// out[b] = ct[b] (.) pt[b]  (pt [level][N]; pt_stride = 0: one plaintext for the batch; a_stride = 0: one ciphertext)
__global__ void __launch_bounds__(256) k_ct_ptmul(const u64* __restrict__ a, size_t a_stride, const u64* __restrict__ pt,
                                                  size_t pt_stride, u64* __restrict__ out, size_t out_stride,
                                                  const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t l = blockIdx.y, bi = blockIdx.z;
    if (c >= N) return;
    const PrimeConst pc = pcs[l];
    const size_t o = (size_t)l * N + c, poly = (size_t)level * N;
    if (!DBG_REGION(pt + bi * pt_stride + o - c, N * sizeof(u64))) return;
    for (int p = 0; p < 2; p++)
        if (!DBG_REGION(a + bi * a_stride + p * poly + o - c, N * sizeof(u64)) || !DBG_REGION(out + bi * out_stride + p * poly + o - c, N * sizeof(u64)))
            return;
    const u64 w = pt[bi * pt_stride + o];
    out[bi * out_stride + o] = mulmod(a[bi * a_stride + o], w, pc);
    out[bi * out_stride + poly + o] = mulmod(a[bi * a_stride + poly + o], w, pc);
}
// keep the first `keep` limbs of a level-`src` ciphertext and multiply them by the integer k
__global__ void __launch_bounds__(256) k_ct_scale_drop(const u64* __restrict__ a, size_t a_stride, u64* __restrict__ out,
                                                       size_t out_stride, const PrimeConst* __restrict__ pcs, uint32_t N,
                                                       uint32_t src, uint32_t keep, u64 k) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t l = blockIdx.y % keep, p = blockIdx.y / keep, bi = blockIdx.z;
    if (c >= N) return;
    const PrimeConst pc = pcs[l];
    const u64 kk = k - mulhi(k, pc.mu) * pc.q;   // k mod q in [0, 2q)
    if (!DBG_REGION(out + bi * out_stride + ((size_t)p * keep + l) * N, N * sizeof(u64)) ||
        !DBG_REGION(a + bi * a_stride + ((size_t)p * src + l) * N, N * sizeof(u64)))
        return;
    out[bi * out_stride + ((size_t)p * keep + l) * N + c] =
        mulmod(a[bi * a_stride + ((size_t)p * src + l) * N + c], csub(kk, pc.q), pc);
}
// multiply by the monomial X^(N/2) `times` times (times = 1: slots * i; times = 3: slots * -i).
// In evaluation order X^(N/2) is I = psi^(N/2) on the first half of the indices and -I on the second.
__global__ void __launch_bounds__(256) k_ct_mul_i(const u64* __restrict__ a, size_t a_stride, u64* __restrict__ out,
                                                  size_t out_stride, const PrimeConst* __restrict__ pcs,
                                                  const ulonglong2* __restrict__ tw, uint32_t N, uint32_t level,
                                                  int times) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t pl = blockIdx.y, bi = blockIdx.z;
    if (c >= N) return;
    const uint32_t l = pl % level;
    const u64 q = pcs[l].q;
    const size_t o = (size_t)pl * N + c;
    if (!DBG_REGION(tw + (size_t)l * N, N * sizeof(ulonglong2)) || !DBG_REGION(a + bi * a_stride + o - c, N * sizeof(u64)) ||
        !DBG_REGION(out + bi * out_stride + o - c, N * sizeof(u64)))
        return;
    const ulonglong2 I = tw[(size_t)l * N + 1];
    u64 v = shoup(a[bi * a_stride + o], I.x, I.y, q);
    const bool neg = (c >= N / 2) != (times == 3);
    out[bi * out_stride + o] = (neg && v) ? q - v : v;
}
// acc += sum over the batch
__global__ void __launch_bounds__(256) k_ct_sum_into(const u64* __restrict__ a, size_t a_stride, uint32_t count,
                                                     u64* __restrict__ acc, const PrimeConst* __restrict__ pcs,
                                                     uint32_t N, uint32_t level) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t pl = blockIdx.y;
    if (c >= N) return;
    const u64 q = pcs[pl % level].q;
    const size_t o = (size_t)pl * N + c;
    if (!DBG_REGION(acc + o - c, N * sizeof(u64))) return;
    for (uint32_t i = 0; i < count; i++)
        if (!DBG_REGION(a + i * a_stride + o - c, N * sizeof(u64))) return;
    u64 s = acc[o];
    for (uint32_t i = 0; i < count; i++) s = addmod(s, a[i * a_stride + o], q);
    acc[o] = s;
}

// out[b] = sum_{j<terms} src_j[b] (.) mask_j on both polynomials (mask_j = masks + j*level*N, shared by the batch);
// the products are summed in 128 bits and reduced once
struct ClassSources {
    const u64* src[16];
};
__global__ void __launch_bounds__(256) k_class_mac(ClassSources s, uint32_t terms, size_t src_stride,
                                                   const u64* __restrict__ masks, u64* __restrict__ out,
                                                   size_t out_stride, const PrimeConst* __restrict__ pcs, uint32_t N,
                                                   uint32_t level) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t l = blockIdx.y, b = blockIdx.z;
    if (c >= N) return;
    const PrimeConst pc = pcs[l];
    const size_t poly = (size_t)level * N, o = (size_t)l * N + c;
    acc128 a0{0, 0}, a1{0, 0};
    for (int p = 0; p < 2; p++)
        if (!DBG_REGION(out + (size_t)b * out_stride + p * poly + o - c, N * sizeof(u64))) return;
    for (uint32_t j = 0; j < terms; j++)
        if (!DBG_REGION(masks + (size_t)j * poly + o - c, N * sizeof(u64)) || !DBG_REGION(s.src[j] + (size_t)b * src_stride + o - c, N * sizeof(u64)) ||
            !DBG_REGION(s.src[j] + (size_t)b * src_stride + poly + o - c, N * sizeof(u64)))
            return;
    for (uint32_t j = 0; j < terms; j++) {
        const u64 w = masks[(size_t)j * poly + o];
        const u64* x = s.src[j] + (size_t)b * src_stride;
        mac128(a0, x[o], w);
        mac128(a1, x[poly + o], w);
    }
    out[(size_t)b * out_stride + o] = reduce128(a0.hi, a0.lo, pc);
    out[(size_t)b * out_stride + poly + o] = reduce128(a1.hi, a1.lo, pc);
}

// ---------------------------------------------------------------------------------------
// host-side sequencing
// ---------------------------------------------------------------------------------------
namespace {

struct Arr {          // `count` compact ciphertexts [2][level][N], `stride` words apart
    u64* p;
    uint32_t count, level;
    size_t stride;
};

struct Geometry {
    uint32_t n, L, H, P, d_s, B, stride, c_state, E, hpc, R, K_s, K_blk, logB, dg;
    uint32_t segs, Bt, dgt;      // token segments of a block (one x / a / output ciphertext each), tokens per segment
    uint32_t l0, l1, lS, linj, lout;
};

static uint32_t ilog2(uint32_t x) {
    uint32_t r = 0;
    while ((1u << (r + 1)) <= x) r++;
    return r;
}

struct Exec {
    fesc_ctx* ctx;
    cudaStream_t st;
    Geometry g;
    const fesc_scan_desc* desc;
    const fesc_scan_consts* cs;
    bool dry;               // planning pass: no launches, only arena accounting
    u64* arena;
    size_t top, high;
    u64* ks;                // key-switch scratch
    u64* rs;                // rescale scratch
    int rc;
    uint32_t N;

    size_t ctw(uint32_t level) const { return (size_t)2 * level * N; }
    Arr alloc(uint32_t count, uint32_t level) {
        Arr a{arena + top, count, level, ctw(level)};
        top += (size_t)count * ctw(level);
        if (top > high) high = top;
        return a;
    }
    Arr at(const Arr& a, uint32_t i, uint32_t count = 1) const { return Arr{a.p + (size_t)i * a.stride, count, a.level, a.stride}; }
    Arr strided(const Arr& a, uint32_t first, uint32_t step, uint32_t count) const {
        return Arr{a.p + (size_t)first * a.stride, count, a.level, a.stride * step};
    }
    bool ok() const { return rc == FESC_OK; }
    dim3 grid(uint32_t rows, uint32_t batch) const { return dim3((N + 255) / 256, rows, batch); }

    uint32_t key_for(int64_t amount) const {
        int64_t n = g.n;
        return desc->key_base + (uint32_t)(((amount % n) + n) % n);
    }
    // out = rot(in, amount)   (amount = slot LEFT shift; in and out must not overlap)
    void rot(const Arr& in, int64_t amount, const Arr& out) {
        if (!ok()) return;
        if (((amount % (int64_t)g.n) + g.n) % g.n == 0) return copy(in, out);
        uint32_t kid = key_for(amount);
        if (!ctx->keys.count(kid)) {
            rc = fesc_fail(ctx, FESC_ENOKEY, "scan_contract: missing Galois key " + std::to_string(kid));
            return;
        }
        if (dry) return;
        rc = rotate_internal(ctx, in.p, in.stride, out.p, out.stride, in.count, in.level, kid, ks, st, 0);
    }
    void conj(const Arr& in, const Arr& out) {
        if (!ok()) return;
        uint32_t kid = desc->key_base + g.n;
        if (!ctx->keys.count(kid)) {
            rc = fesc_fail(ctx, FESC_ENOKEY, "scan_contract: missing conjugation key");
            return;
        }
        if (dry) return;
        rc = rotate_internal(ctx, in.p, in.stride, out.p, out.stride, in.count, in.level, kid, ks, st, 0);
    }
    void copy(const Arr& in, const Arr& out) {
        if (!ok() || dry || in.p == out.p) return;
        size_t w = ctw(in.level) * sizeof(u64);
        cudaError_t e = cudaMemcpy2DAsync(out.p, out.stride * sizeof(u64), in.p, in.stride * sizeof(u64), w, in.count,
                                          cudaMemcpyDeviceToDevice, st);
        if (e != cudaSuccess) rc = fesc_fail(ctx, FESC_ECUDA, cudaGetErrorString(e));
    }
    void addsub(const Arr& a, const Arr& b, const Arr& out, int sub) {
        if (!ok() || dry) return;
        prof_begin(ctx, PF_POINTWISE, st);
        k_ct_addsub<<<grid(2 * a.level, a.count), 256, 0, st>>>(a.p, a.stride, b.p, b.count == 1 && a.count > 1 ? 0 : b.stride,
                                                                out.p, out.stride, ctx->d_pc, N, a.level, sub);
        prof_end(ctx, PF_POINTWISE, st);
    }
    void add(const Arr& a, const Arr& b, const Arr& out) { addsub(a, b, out, 0); }
    void sub(const Arr& a, const Arr& b, const Arr& out) { addsub(a, b, out, 1); }
    void mul_i(const Arr& a, const Arr& out, int times) {
        if (!ok() || dry) return;
        prof_begin(ctx, PF_POINTWISE, st);
        k_ct_mul_i<<<grid(2 * a.level, a.count), 256, 0, st>>>(a.p, a.stride, out.p, out.stride, ctx->d_pc, ctx->d_tw, N,
                                                               a.level, times);
        prof_end(ctx, PF_POINTWISE, st);
    }
    // contiguous `in` at level l -> contiguous `out` at level l-1
    void rescale(const Arr& in, const Arr& out) {
        if (!ok() || dry) return;
        rc = rescale_internal(ctx, in.p, in.stride, out.p, in.count, in.level, rs, st);
    }
    // out (level-1, contiguous) = rescale(in (.) pt); pt_stride != 0: plaintext i for element i; a single `in` with
    // out.count plaintexts multiplies that one ciphertext by each of them
    void ptmul_rescale(const Arr& in, const u64* pt, const Arr& out, size_t pt_stride = 0) {
        size_t mark = top;
        const uint32_t cnt = out.count;
        Arr t = alloc(cnt, in.level);
        if (ok() && !dry) {
            prof_begin(ctx, PF_POINTWISE, st);
            k_ct_ptmul<<<grid(in.level, cnt), 256, 0, st>>>(in.p, in.count == 1 && cnt > 1 ? 0 : in.stride, pt, pt_stride, t.p,
                                                            t.stride, ctx->d_pc, N, in.level);
            prof_end(ctx, PF_POINTWISE, st);
            ctx->counters[2] += cnt;
        }
        rescale(t, out);
        top = mark;
    }
    // out (level-1, contiguous) = rescale(a * b); b may be a single ciphertext shared by the batch
    void mul_rescale(const Arr& a, const Arr& b, const Arr& out) {
        size_t mark = top;
        Arr t = alloc(a.count, a.level);
        if (ok() && !dry)
            rc = ctmul_internal(ctx, a.p, a.stride, b.p, (b.count == 1 && a.count > 1) ? 0 : b.stride, t.p, t.stride, a.count,
                                a.level, ks, st);
        rescale(t, out);
        top = mark;
    }
    // out (level dst, contiguous) = in brought from its level to dst; kind 0: state-like, 1: multiplicand
    void adjust(const Arr& in, uint32_t dst, int kind, const Arr& out) {
        if (!ok()) return;
        if (in.level == dst) return copy(in, out);
        if (in.level < dst) {
            rc = fesc_fail(ctx, FESC_ELEVEL, "scan_contract: level schedule violated");
            return;
        }
        size_t mark = top;
        Arr t = alloc(in.count, dst + 1);
        if (!dry) {
            const uint64_t* tab = kind ? cs->adj_p : cs->adj_s;
            u64 k = tab[(size_t)in.level * (g.l0 + 1) + dst];
            prof_begin(ctx, PF_POINTWISE, st);
            k_ct_scale_drop<<<grid(2 * (dst + 1), in.count), 256, 0, st>>>(in.p, in.stride, t.p, t.stride, ctx->d_pc, N,
                                                                           in.level, dst + 1, k);
            prof_end(ctx, PF_POINTWISE, st);
        }
        rescale(t, out);
        top = mark;
    }
    // out[i] (level dst, contiguous) = slot pos[i] of `base` (capacity stride base.stride, current level lev[pos[i]])
    // brought to dst.  Slots that sit at the same level go down in ONE batch: straight from the slots when their
    // positions are equally spaced, through a gathered copy otherwise; the result lands in out directly when the
    // group is a run of consecutive outputs.
    void adjust_many(const Arr& base, const std::vector<uint32_t>& pos, const std::vector<uint32_t>& lev, uint32_t dst,
                     int kind, const Arr& out) {
        std::map<uint32_t, std::vector<uint32_t>> groups;      // source level -> output indices
        for (uint32_t i = 0; i < pos.size(); i++) groups[lev[pos[i]]].push_back(i);
        for (auto& kv : groups) {
            const uint32_t src = kv.first;
            const std::vector<uint32_t>& idx = kv.second;
            const uint32_t cnt = (uint32_t)idx.size();
            auto slot = [&](uint32_t i) { return Arr{base.p + (size_t)pos[i] * base.stride, 1, src, ctw(src)}; };
            if (src == dst || cnt == 1) {
                for (uint32_t i : idx) adjust(slot(i), dst, kind, at(out, i));
                continue;
            }
            bool spaced = true, run = true;
            const int64_t step = (int64_t)pos[idx[1]] - (int64_t)pos[idx[0]];
            for (uint32_t k = 1; k < cnt; k++) {
                spaced = spaced && step > 0 && (int64_t)pos[idx[k]] - (int64_t)pos[idx[k - 1]] == step;
                run = run && idx[k] == idx[k - 1] + 1;
            }
            size_t mark = top;
            Arr gin = spaced ? Arr{base.p + (size_t)pos[idx[0]] * base.stride, cnt, src, base.stride * (size_t)step}
                             : alloc(cnt, src);
            if (!spaced)
                for (uint32_t k = 0; k < cnt; k++) copy(slot(idx[k]), at(gin, k));
            if (run) {
                adjust(gin, dst, kind, at(out, idx[0], cnt));
            } else {
                Arr gout = alloc(cnt, dst);
                adjust(gin, dst, kind, gout);
                for (uint32_t k = 0; k < cnt; k++) copy(at(gout, k), at(out, idx[k]));
            }
            top = mark;
        }
    }
    bool key_ok(int64_t amount) {
        uint32_t kid = key_for(amount);
        if (ctx->keys.count(kid)) return true;
        rc = fesc_fail(ctx, FESC_ENOKEY, "scan_contract: missing Galois key " + std::to_string(kid));
        return false;
    }
    // a += rot(a, unit * 2^b) for b = 0..steps-1 (unit signed).  Hoisted mode takes steps (b, b+1) together:
    // a + rot(a, d) + rot(a, 2d) + rot(a, 3d), d = unit * 2^b, with one decomposition and one division by P.
    void chain(const Arr& a, int64_t unit, uint32_t steps) {
        size_t mark = top;
        Arr t = alloc(a.count, a.level);
        uint32_t b = 0;
        while (b < steps && ok()) {
            const int64_t d = unit * (int64_t)(1u << b);
            if (desc->hoist && b + 1 < steps) {
                if (!key_ok(d) || !key_ok(2 * d) || !key_ok(3 * d)) break;
                if (!dry) {
                    const uint32_t ids[3] = {key_for(d), key_for(2 * d), key_for(3 * d)};
                    rc = rotate_sum_hoisted_internal(ctx, a.p, a.stride, t.p, t.stride, a.count, a.level, ids, 3, ks, st);
                    copy(t, a);
                }
                b += 2;
            } else {
                rot(a, d, t);
                add(a, t, a);
                b += 1;
            }
        }
        top = mark;
    }
    void fill_right(const Arr& a, uint32_t unit, uint32_t steps) { chain(a, -(int64_t)unit, steps); }
    // Broadcasts of the tokens of filled group ciphertexts (grouped leaf build): for class c < G
    //   out_c[u] = rescale( sum_{j<G} masks[j] (.) rot(grp[u], (c - j) unit) ),
    // with the 2(G-1) rotations by +unit..+(G-1)unit, -unit..-(G-1)unit taken once for the whole batch of groups
    // (hoisted mode: one decomposition per group).  `deliver(c, res)` receives the batch of class c (level - 1,
    // contiguous, valid until it returns).
    template <class F>
    void class_broadcasts(const Arr& grp, const u64* masks, uint32_t G, uint32_t unit, F deliver) {
        size_t mark = top;
        const uint32_t nk = 2 * (G - 1), cnt = grp.count, lvl = grp.level;
        Arr rots = alloc(nk * cnt, lvl);       // [shift][group]
        std::vector<int64_t> shifts;
        for (uint32_t k = 1; k < G; k++) shifts.push_back((int64_t)k * unit);
        for (uint32_t k = 1; k < G; k++) shifts.push_back(-(int64_t)k * unit);
        if (desc->hoist) {
            std::vector<uint32_t> ids;
            for (int64_t d : shifts)
                if (key_ok(d)) ids.push_back(key_for(d));
            if (ok() && !dry)
                rc = rotate_hoisted_internal(ctx, grp.p, grp.stride, rots.p, rots.stride, (size_t)cnt * rots.stride, cnt, lvl,
                                             ids.data(), nk, ks, st);
        } else {
            for (uint32_t i = 0; i < nk; i++) rot(grp, shifts[i], at(rots, i * cnt, cnt));
        }
        Arr acc = alloc(cnt, lvl), res = alloc(cnt, lvl - 1);
        for (uint32_t c = 0; c < G && ok(); c++) {
            if (!dry) {
                ClassSources cs_;
                for (uint32_t j = 0; j < G; j++) {
                    const int k = (int)c - (int)j;
                    cs_.src[j] = k == 0 ? grp.p : rots.p + (size_t)(k > 0 ? k - 1 : (int)G - 2 - k) * cnt * rots.stride;
                }
                prof_begin(ctx, PF_POINTWISE, st);
                k_class_mac<<<grid(lvl, cnt), 256, 0, st>>>(cs_, G, grp.stride, masks, acc.p, acc.stride, ctx->d_pc, N, lvl);
                prof_end(ctx, PF_POINTWISE, st);
                ctx->counters[2] += (uint64_t)G * cnt;
            }
            rescale(acc, res);
            deliver(c, res);
        }
        top = mark;
    }
    // out[t] = rot(src, unit * t) for t = 0..count-1, via t = t_lo + dg * t_hi, dg = min(16, count) (hoisted mode:
    // the dg-1 low-digit rotations of one ciphertext share its decomposition)
    void extract_n(const Arr& src, int64_t unit, uint32_t count, const Arr& out) {
        size_t mark = top;
        const uint32_t dg = count < 16 ? count : 16, nh = count / dg;
        Arr gi = alloc(nh, src.level);
        for (uint32_t th = 0; th < nh; th++) rot(src, unit * (int64_t)(dg * th), at(gi, th));
        if (desc->hoist && dg > 1) {
            copy(gi, strided(out, 0, dg, nh));
            std::vector<uint32_t> ids;
            for (uint32_t tl = 1; tl < dg && ok(); tl++)
                if (key_ok(unit * (int64_t)tl)) ids.push_back(key_for(unit * (int64_t)tl));
            if (ok() && !dry)
                rc = rotate_hoisted_internal(ctx, gi.p, gi.stride, out.p + out.stride, out.stride * dg, out.stride, nh,
                                             src.level, ids.data(), (uint32_t)ids.size(), ks, st);
        } else {
            for (uint32_t tl = 0; tl < dg; tl++) rot(gi, unit * (int64_t)tl, strided(out, tl, dg, nh));
        }
        top = mark;
    }
    void extract_all(const Arr& src, int64_t unit, const Arr& out) { extract_n(src, unit, g.B, out); }
};

}  // namespace

static int scan_run(Exec& X, const u64* d_x, const u64* d_a, const u64* d_B, const u64* d_C, u64* d_out) {
    const Geometry& g = X.g;
    const uint32_t B = g.B, l0 = g.l0, l1 = g.l1, lS = g.lS, linj = g.linj, lout = g.lout;
    const uint32_t N = X.N;
    const size_t in_ctw = X.ctw(l0), out_ctw = X.ctw(lout);
    if (!X.dry) {
        cudaError_t e = cudaMemsetAsync(d_out, 0, (size_t)g.K_blk * g.K_s * g.segs * out_ctw * sizeof(u64), X.st);
        if (e != cudaSuccess) return fesc_fail(X.ctx, FESC_ECUDA, cudaGetErrorString(e));
    }
    // carries g_j per chunk (level lS - (j-1)), stored at capacity lS
    Arr carry = X.alloc(g.K_s, lS);
    std::vector<uint32_t> carry_level(g.K_s, 0);
    for (uint32_t j = 0; j < g.K_blk && X.ok(); j++) {
        const size_t block_mark = X.top;
        // ---- br(B_t) at l0-1 (l0-2 with the grouped leaf build) and br(C_t) at linj-1, shared by every chunk ----
        const uint32_t G = X.desc->group, lB = G ? l0 - 2 : l0 - 1;
        const bool plain = X.desc->plain != 0;      // invariant families: plaintext decay, B and C; nothing to broadcast
        const size_t row0 = (size_t)l0 * N;         // pitch of the plaintext tables that hold one level per row
        Arr brB = X.alloc(plain ? 0 : B, lB), brC = X.alloc(plain ? 0 : B, linj - 1);
        for (int which = 0; which < 2 && !plain; which++) {
            size_t m = X.top;
            Arr src{const_cast<u64*>((which ? d_C : d_B) + (size_t)j * in_ctw), 1, l0, in_ctw};
            if (which == 0 && G) {
                // br(B_t) for groups of G tokens (G d_s consecutive slots): one extraction, mask and fill per group,
                // then every token as a masked sum of the group's rotations by multiples of d_s; lands at l0-2
                const uint32_t ng = B / G, unit = G * g.d_s;
                Arr exg = X.alloc(ng, l0), gb = X.alloc(ng, l0 - 1);
                X.extract_n(src, unit, ng, exg);
                X.ptmul_rescale(exg, (const u64*)X.cs->d_mask_bg, gb);
                X.fill_right(gb, unit, ilog2(g.n / unit));
                X.class_broadcasts(gb, (const u64*)X.cs->d_mask_b2, G, g.d_s,
                                   [&](uint32_t c, const Arr& res) { X.copy(res, X.strided(brB, c, G, ng)); });
                X.top = m;
                continue;
            }
            Arr ex = X.alloc(B, l0);
            X.extract_all(src, g.d_s, ex);
            if (which == 0) {
                X.ptmul_rescale(ex, (const u64*)X.cs->d_mask_b, brB);
                X.fill_right(brB, g.stride, ilog2(g.c_state));
            } else {
                // br(C) is only needed at the injection level: bring it down first, fill there (cheap rotations)
                Arr full = X.alloc(B, l0 - 1);
                X.ptmul_rescale(ex, (const u64*)X.cs->d_mask_b, full);
                X.adjust(full, linj - 1, 1, brC);
                X.fill_right(brC, g.stride, ilog2(g.c_state));
            }
            X.top = m;
        }
        // contracted products of the block, [chunk parity][token], level linj-2
        Arr V = X.alloc(2 * B, linj - 2);
        for (uint32_t kap = 0; kap < g.K_s && X.ok(); kap++) {
            const size_t chunk_mark = X.top;
            // position slots of the prefix network: capacity l1, current level tracked on the host
            Arr Ps = X.alloc(plain ? 0 : B, l1), Ss = X.alloc(B, l1);
            std::vector<uint32_t> lp(B, l1), ls(B, l1);
            if (plain) {   // ---- leaves of the invariant families: s_t = br(x_t) (.) Bbar, no decay component ----
                size_t m = X.top;
                const size_t seg0 = ((size_t)j * g.K_s + kap) * g.segs;
                Arr srcx{const_cast<u64*>(d_x + seg0 * in_ctw), g.segs, l0, in_ctw};
                Arr xr = X.alloc(B, lB);
                if (G) {
                    const uint32_t ng = B / G, ngs = g.Bt / G;
                    Arr ex = X.alloc(ng, l0), xg = X.alloc(ng, l0 - 1);
                    for (uint32_t sg = 0; sg < g.segs; sg++) X.extract_n(X.at(srcx, sg), G, ngs, X.at(ex, sg * ngs, ngs));
                    X.ptmul_rescale(ex, (const u64*)X.cs->d_mask_xg, xg);
                    X.fill_right(xg, G, ilog2(g.d_s / G));
                    X.class_broadcasts(xg, (const u64*)X.cs->d_mask_x2, G, 1,
                                       [&](uint32_t c, const Arr& res) { X.copy(res, X.strided(xr, c, G, ng)); });
                } else {
                    Arr ex = X.alloc(B, l0);
                    for (uint32_t sg = 0; sg < g.segs; sg++) X.extract_n(X.at(srcx, sg), 1, g.Bt, X.at(ex, sg * g.Bt, g.Bt));
                    X.ptmul_rescale(ex, (const u64*)X.cs->d_mask_x, xr);
                    X.fill_right(xr, 1, ilog2(g.d_s));
                }
                X.ptmul_rescale(xr, (const u64*)X.cs->d_pt_b, Ss);
                X.top = m;
            } else if (G) {   // ---- leaves, grouped build: groups of G tokens share extraction, mask and fill ----
                size_t m = X.top;
                const uint32_t ng = B / G, ngs = g.Bt / G;      // groups per block / per segment
                const size_t seg0 = ((size_t)j * g.K_s + kap) * g.segs;
                Arr srcx{const_cast<u64*>(d_x + seg0 * in_ctw), g.segs, l0, in_ctw};
                Arr apre = X.alloc(g.segs, l0);
                X.copy(Arr{const_cast<u64*>(d_a + seg0 * in_ctw), g.segs, l0, in_ctw}, apre);
                X.fill_right(apre, 1, ilog2(g.P));
                Arr ex = X.alloc(ng, l0), xg = X.alloc(ng, l0 - 1), ag = X.alloc(ng, l0 - 1);
                for (uint32_t sg = 0; sg < g.segs; sg++) X.extract_n(X.at(srcx, sg), G, ngs, X.at(ex, sg * ngs, ngs));
                X.ptmul_rescale(ex, (const u64*)X.cs->d_mask_xg, xg);
                X.fill_right(xg, G, ilog2(g.d_s / G));
                for (uint32_t sg = 0; sg < g.segs; sg++)
                    X.extract_n(X.at(apre, sg), (int64_t)G * g.P, ngs, X.at(ex, sg * ngs, ngs));
                X.ptmul_rescale(ex, (const u64*)X.cs->d_mask_ag, ag);
                X.fill_right(ag, G * g.P, ilog2(g.R / (G * g.P)));
                Arr xr = X.alloc(B, l0 - 2), cls1 = X.alloc(ng, l1);
                // class c = the tokens u*G + c of every group u
                X.class_broadcasts(xg, (const u64*)X.cs->d_mask_x2, G, 1,
                                   [&](uint32_t c, const Arr& res) { X.copy(res, X.strided(xr, c, G, ng)); });
                X.class_broadcasts(ag, (const u64*)X.cs->d_mask_a2, G, g.P, [&](uint32_t c, const Arr& res) {
                    X.adjust(res, l1, 1, cls1);          // p_t = br(a_t) at the leaf level
                    X.copy(cls1, X.strided(Ps, c, G, ng));
                });
                X.mul_rescale(xr, brB, Ss);      // s_t = br(x_t) (.) br(B_t), level l1 = l0-3
                X.top = m;
            } else {   // ---- leaves ----
                size_t m = X.top;
                const size_t seg0 = ((size_t)j * g.K_s + kap) * g.segs;
                Arr srcx{const_cast<u64*>(d_x + seg0 * in_ctw), g.segs, l0, in_ctw};
                Arr apre = X.alloc(g.segs, l0);
                X.copy(Arr{const_cast<u64*>(d_a + seg0 * in_ctw), g.segs, l0, in_ctw}, apre);
                X.fill_right(apre, 1, ilog2(g.P));
                Arr ex = X.alloc(B, l0), xr = X.alloc(B, l0 - 1), ar = X.alloc(B, l0 - 1);
                for (uint32_t sg = 0; sg < g.segs; sg++) X.extract_n(X.at(srcx, sg), 1, g.Bt, X.at(ex, sg * g.Bt, g.Bt));
                X.ptmul_rescale(ex, (const u64*)X.cs->d_mask_x, xr);
                X.fill_right(xr, 1, ilog2(g.d_s));
                for (uint32_t sg = 0; sg < g.segs; sg++) X.extract_n(X.at(apre, sg), g.P, g.Bt, X.at(ex, sg * g.Bt, g.Bt));
                X.ptmul_rescale(ex, (const u64*)X.cs->d_mask_a, ar);
                X.adjust(ar, l1, 1, Ps);         // p_t = br(a_t): to the leaf level first, then the fill
                X.fill_right(Ps, g.P, ilog2(g.R / g.P));
                X.mul_rescale(xr, brB, Ss);      // s_t = br(x_t) (.) br(B_t), level l1 (slots are compact at l1)
                X.top = m;
            }
            // ---- Brent-Kung network ----
            // one stage: nodes (left position, right position), operands brought to `lvl`, results at lvl-1
            const u64* stage_pt = nullptr;          // invariant families: abar^span at the stage's level
            auto stage = [&](const std::vector<uint32_t>& left, const std::vector<uint32_t>& right, uint32_t lvl, bool need_p) {
                const uint32_t cnt = (uint32_t)left.size();
                if (!cnt || !X.ok()) return;
                size_t m = X.top;
                if (plain) {        // s <- abar^span (.) s_L + s_R: one ct-pt product per node
                    Arr sL = X.alloc(cnt, lvl), sR = X.alloc(cnt, lvl - 1), ns = X.alloc(cnt, lvl - 1);
                    X.adjust_many(Ss, left, ls, lvl, 0, sL);
                    X.adjust_many(Ss, right, ls, lvl - 1, 0, sR);
                    X.ptmul_rescale(sL, stage_pt, ns);
                    X.add(ns, sR, ns);
                    for (uint32_t i = 0; i < cnt; i++) {
                        const uint32_t b = right[i];
                        X.copy(X.at(ns, i), Arr{Ss.p + (size_t)b * Ss.stride, 1, lvl - 1, X.ctw(lvl - 1)});
                        ls[b] = lvl - 1;
                    }
                    X.top = m;
                    return;
                }
                Arr pL = X.alloc(cnt, lvl), sL = X.alloc(cnt, lvl), pR = X.alloc(cnt, lvl), sR = X.alloc(cnt, lvl - 1);
                Arr np_ = X.alloc(cnt, lvl - 1), ns = X.alloc(cnt, lvl - 1);
                if (need_p) X.adjust_many(Ps, left, lp, lvl, 1, pL);
                X.adjust_many(Ss, left, ls, lvl, 0, sL);
                X.adjust_many(Ps, right, lp, lvl, 1, pR);
                X.adjust_many(Ss, right, ls, lvl - 1, 0, sR);
                if (need_p) X.mul_rescale(pR, pL, np_);
                X.mul_rescale(pR, sL, ns);
                X.add(ns, sR, ns);
                for (uint32_t i = 0; i < cnt; i++) {
                    const uint32_t b = right[i];
                    if (need_p) {
                        X.copy(X.at(np_, i), Arr{Ps.p + (size_t)b * Ps.stride, 1, lvl - 1, X.ctw(lvl - 1)});
                        lp[b] = lvl - 1;
                    }
                    X.copy(X.at(ns, i), Arr{Ss.p + (size_t)b * Ss.stride, 1, lvl - 1, X.ctw(lvl - 1)});
                    ls[b] = lvl - 1;
                }
                X.top = m;
            };
            const uint32_t network = X.desc->network;
            for (uint32_t s = 1; s <= g.logB; s++) {
                std::vector<uint32_t> left, right;
                const uint32_t half = 1u << (s - 1);
                if (network == FESC_NET_KOGGE_STONE) {          // every k > 2^(s-1) with k - 2^(s-1) (1-based)
                    for (uint32_t k = half + 1; k <= B; k++) {
                        left.push_back(k - half - 1);
                        right.push_back(k - 1);
                    }
                } else if (network == FESC_NET_SKLANSKY) {      // upper half of every block of 2^s with the lower half's last
                    for (uint32_t b = 0; b < (B >> s); b++)
                        for (uint32_t k = (b << s) + half; k < ((b + 1) << s); k++) {
                            left.push_back((b << s) + half - 1);
                            right.push_back(k);
                        }
                } else {
                    for (uint32_t k = 1u << s; k <= B; k += 1u << s) {
                        left.push_back(k - half - 1);
                        right.push_back(k - 1);
                    }
                }
                // the last stage of a one-pass network forms decay products only for an incoming state
                if (plain) stage_pt = (const u64*)X.cs->d_pt_up + (size_t)(s - 1) * row0;
                stage(left, right, l1 - (s - 1), network == FESC_NET_BRENT_KUNG || s < g.logB || j > 0);
            }
            // summary of the block = last position after the up-sweep (after the last stage of a one-pass network);
            // keep a copy for the carry (the first block's decay product is not used)
            Arr sumP = X.alloc(1, lS), sumS = X.alloc(1, lS);
            if (!plain && (network == FESC_NET_BRENT_KUNG || j > 0)) X.copy(Arr{Ps.p + (size_t)(B - 1) * Ps.stride, 1, lS, X.ctw(lS)}, sumP);
            X.copy(Arr{Ss.p + (size_t)(B - 1) * Ss.stride, 1, lS, X.ctw(lS)}, sumS);
            uint32_t d = 0;
            for (uint32_t s = g.logB - 1; s >= 1 && network == FESC_NET_BRENT_KUNG; s--) {
                d++;
                std::vector<uint32_t> left, right;
                for (uint32_t k = 1u << s; k < B; k += 1u << s) {
                    uint32_t r = k + (1u << (s - 1));
                    if (r < B) {
                        left.push_back(k - 1);
                        right.push_back(r - 1);
                    }
                }
                if (plain) stage_pt = (const u64*)X.cs->d_pt_down + (size_t)(d - 1) * row0;
                stage(left, right, lS - (d - 1), j > 0);
            }
            // ---- carry injection and contraction with br(C_t) ----
            {
                size_t m = X.top;
                Arr h = X.alloc(B, linj - 1);
                std::vector<uint32_t> every(B);
                for (uint32_t t = 0; t < B; t++) every[t] = t;
                X.adjust_many(Ss, every, ls, linj - 1, 0, h);
                if (j > 0) {
                    Arr pp = X.alloc(plain ? 0 : B, linj), gg = X.alloc(1, linj), pg = X.alloc(B, linj - 1);
                    X.adjust(Arr{carry.p + (size_t)kap * carry.stride, 1, carry_level[kap], X.ctw(carry_level[kap])}, linj, 0, gg);
                    if (plain) {    // state_t = abar^(t+1) (.) g_j + s_t
                        X.ptmul_rescale(gg, (const u64*)X.cs->d_pt_inj, pg, (size_t)linj * N);
                    } else {
                        X.adjust_many(Ps, every, lp, linj, 1, pp);
                        X.mul_rescale(pp, gg, pg);
                    }
                    X.add(h, pg, h);
                }
                if (plain) X.ptmul_rescale(h, (const u64*)X.cs->d_pt_c, X.at(V, (kap & 1) * B, B));
                else X.mul_rescale(h, brC, X.at(V, (kap & 1) * B, B));
                X.top = m;
            }
            // ---- serialized carry g_{j+1} = S_j(g_j) ----
            if (j + 1 < g.K_blk) {
                Arr slot{carry.p + (size_t)kap * carry.stride, 1, 0, 0};
                if (j == 0) {
                    slot.level = lS;
                    slot.stride = X.ctw(lS);
                    X.copy(sumS, slot);
                    carry_level[kap] = lS;
                } else {
                    const uint32_t lg = carry_level[kap];
                    size_t m = X.top;
                    Arr gcur{slot.p, 1, lg, X.ctw(lg)};
                    Arr pa = X.alloc(1, lg), sa = X.alloc(1, lg - 1), ng = X.alloc(1, lg - 1);
                    X.adjust(sumS, lg - 1, 0, sa);
                    if (plain) {    // g_{j+1} = abar^B (.) g_j + s_S
                        X.ptmul_rescale(gcur, (const u64*)X.cs->d_pt_carry + (size_t)j * row0, ng);
                    } else {
                        X.adjust(sumP, lg, 1, pa);
                        X.mul_rescale(pa, gcur, ng);
                    }
                    X.add(ng, sa, ng);
                    X.copy(ng, Arr{slot.p, 1, lg - 1, X.ctw(lg - 1)});
                    carry_level[kap] = lg - 1;
                    X.top = m;
                }
            }
            X.top = chunk_mark;
            // ---- state-axis reduction of a chunk pair (or of the unpaired last chunk) ----
            const bool second = (kap & 1) != 0, last = kap + 1 == g.K_s;
            if (second || last) {
                const bool paired = second;
                const uint32_t k0 = paired ? kap - 1 : kap;
                const uint32_t lred = linj - 2;
                size_t m = X.top;
                Arr chi = X.alloc(B, lred), tmp = X.alloc(B, lred);
                Arr v0 = X.at(V, (k0 & 1) * B, B), v1 = X.at(V, ((k0 + 1) & 1) * B, B);
                if (paired) {
                    X.mul_i(v1, tmp, 1);
                    X.add(v0, tmp, chi);
                } else {
                    X.copy(v0, chi);
                }
                X.chain(chi, 1, ilog2(g.d_s));
                Arr part = X.alloc(B, lred), y = X.alloc(B, lout), y2 = X.alloc(B, lout);
                const uint32_t nparts = paired ? 2 : 1;
                if (paired) X.conj(chi, tmp);
                for (uint32_t which = 0; which < nparts; which++) {
                    if (!paired) {
                        X.add(chi, chi, part);
                    } else if (which == 0) {
                        X.add(chi, tmp, part);                 // 2 Re
                    } else {
                        X.sub(chi, tmp, part);
                        X.mul_i(part, part, 3);                // -i (Xi - conj Xi) = 2 Im
                    }
                    X.ptmul_rescale(part, (const u64*)X.cs->d_mask_out, y);
                    // placement: rotate right by the offset inside the token's segment, t' = t_lo + dgt * t_hi
                    // (t = seg*Bt + t' and dgt divides Bt, so t mod dgt = t_lo and the high digit is (t / dgt) mod (Bt / dgt))
                    const uint32_t nh = B / g.dgt, nhs = g.Bt / g.dgt;
                    for (uint32_t tl = 0; tl < g.dgt; tl++)
                        X.rot(X.strided(y, tl, g.dgt, nh), -(int64_t)tl, X.strided(y2, tl, g.dgt, nh));
                    for (uint32_t th = 0; th < nh; th++)
                        X.rot(X.at(y2, th * g.dgt, g.dgt), -(int64_t)(g.dgt * (th % nhs)), X.at(y, th * g.dgt, g.dgt));
                    for (uint32_t sg = 0; sg < g.segs && X.ok() && !X.dry; sg++) {
                        u64* dst = d_out + (((size_t)j * g.K_s + k0 + which) * g.segs + sg) * out_ctw;
                        prof_begin(X.ctx, PF_POINTWISE, X.st);
                        k_ct_sum_into<<<dim3((N + 255) / 256, 2 * lout), 256, 0, X.st>>>(y.p + (size_t)sg * g.Bt * y.stride, y.stride,
                                                                                         g.Bt, dst, X.ctx->d_pc, N, lout);
                        prof_end(X.ctx, PF_POINTWISE, X.st);
                    }
                }
                X.top = m;
            }
        }
        X.top = block_mark;
    }
    return X.rc;
}

extern "C" int fesc_scan_contract(fesc_ctx* ctx, const uint64_t* d_x, const uint64_t* d_a, const uint64_t* d_B,
                                  const uint64_t* d_C, const fesc_scan_desc* desc, const fesc_scan_consts* consts,
                                  uint64_t* d_m_out, void* stream) {
    if (!ctx || !d_x || !desc || !consts || !d_m_out) return FESC_EINVAL;
    const bool plain = desc->plain != 0;
    if (!plain && (!d_a || !d_B || !d_C)) return FESC_EINVAL;
    if (!consts->d_mask_x || !consts->d_mask_out || !consts->adj_s || (!plain && (!consts->d_mask_a || !consts->d_mask_b || !consts->adj_p)))
        return fesc_fail(ctx, FESC_EINVAL, "scan_contract: missing constants");
    if (plain && desc->network != FESC_NET_BRENT_KUNG)
        return fesc_fail(ctx, FESC_EINVAL, "scan_contract: the invariant-family mode uses the Brent-Kung schedule");
    Geometry g;
    g.n = ctx->N / 2;
    g.L = desc->L, g.H = desc->H, g.P = desc->P, g.d_s = desc->d_s, g.B = desc->B_blk;
    auto pow2 = [](uint32_t v) { return v && !(v & (v - 1)); };
    if (!g.L || !g.H || !pow2(g.P) || !pow2(g.d_s) || !pow2(g.B) || g.B < 2)
        return fesc_fail(ctx, FESC_EINVAL, "scan_contract: P, d_s, B_blk must be powers of two, B_blk >= 2");
    g.stride = desc->stride ? desc->stride : (g.d_s > g.B ? g.d_s : g.B);
    if (!pow2(g.stride) || g.stride < g.d_s || g.stride > g.n)
        return fesc_fail(ctx, FESC_EINVAL, "scan_contract: bad stride");
    g.segs = g.B > g.stride ? g.B / g.stride : 1;
    g.Bt = g.B / g.segs;
    g.dgt = g.Bt < 16 ? g.Bt : 16;
    g.c_state = g.n / g.stride;
    g.E = g.H * g.P;
    if (g.c_state % g.P || g.E % g.c_state) return fesc_fail(ctx, FESC_EINVAL, "scan_contract: channels do not tile the chunks");
    g.hpc = g.c_state / g.P;
    g.R = g.n / g.hpc;
    g.K_s = g.E / g.c_state;
    g.K_blk = (g.L + g.B - 1) / g.B;
    g.logB = ilog2(g.B);
    g.dg = g.B < 16 ? g.B : 16;
    if ((uint64_t)g.B * g.d_s > g.n || (uint64_t)g.Bt * g.P > g.R)
        return fesc_fail(ctx, FESC_EINVAL, "scan_contract: block does not fit the compact packings");
    g.l0 = desc->n_limbs;
    if (desc->network > FESC_NET_SKLANSKY) return fesc_fail(ctx, FESC_EINVAL, "scan_contract: unknown prefix network");
    const uint32_t below_summary =
        desc->network == FESC_NET_BRENT_KUNG ? g.logB - 1 : (g.K_blk > 2 ? g.K_blk - 2 : 0);   // lS - linj
    const uint32_t G = desc->group;
    if (G) {
        if (G < 2 || (G & (G - 1)) || G > 16 || G > g.Bt || G > g.d_s)
            return fesc_fail(ctx, FESC_EINVAL, "scan_contract: group must be a power of two, at most 16, the tokens of a segment and d_s");
        if (!consts->d_mask_xg || !consts->d_mask_x2 ||
            (!plain && (!consts->d_mask_ag || !consts->d_mask_a2 || !consts->d_mask_bg || !consts->d_mask_b2)))
            return fesc_fail(ctx, FESC_EINVAL, "scan_contract: the grouped leaf build needs its mask arrays");
    }
    if (g.l0 > ctx->n_q || g.l0 < g.logB + below_summary + 6 + (G ? 1 : 0))
        return fesc_fail(ctx, FESC_ELEVEL, "scan_contract: not enough levels");
    g.l1 = g.l0 - (G ? 3 : 2);
    g.lS = g.l1 - g.logB;
    g.linj = g.lS - below_summary;
    g.lout = g.linj - 3;
    if (g.K_blk > 1 && g.lS < g.linj + (g.K_blk - 2))
        return fesc_fail(ctx, FESC_ELEVEL, "scan_contract: carry chain runs below the injection level");
    if (plain && (!consts->d_pt_b || !consts->d_pt_c || !consts->d_pt_up || (g.logB > 1 && !consts->d_pt_down) ||
                  (g.K_blk > 1 && !consts->d_pt_inj) || (g.K_blk > 2 && !consts->d_pt_carry)))
        return fesc_fail(ctx, FESC_EINVAL, "scan_contract: the invariant-family mode needs its plaintext tables");
    Exec X;
    X.ctx = ctx, X.st = (cudaStream_t)stream, X.g = g, X.desc = desc, X.cs = consts;
    X.N = ctx->N, X.rc = FESC_OK;
    // planning pass for the arena size
    X.dry = true, X.arena = reinterpret_cast<u64*>((uintptr_t)1 << 40), X.top = 0, X.high = 0, X.ks = X.rs = nullptr;
    int rc = scan_run(X, (const u64*)d_x, (const u64*)d_a, (const u64*)d_B, (const u64*)d_C, (u64*)d_m_out);
    if (rc != FESC_OK) return rc;
    const size_t ks_words = ks_scratch_words(ctx, g.l0, ks_chunk(ctx, 2 * g.B));
    const size_t rs_words = (size_t)2 * g.B * 2 * ctx->N;
    u64* scratch;
    rc = ctx_scratch(ctx, (X.high + ks_words + rs_words) * sizeof(u64), &scratch);
    if (rc != FESC_OK) return rc;
    X.dry = false, X.arena = scratch, X.top = 0;
    X.ks = scratch + X.high;
    X.rs = X.ks + ks_words;
    return scan_run(X, (const u64*)d_x, (const u64*)d_a, (const u64*)d_B, (const u64*)d_C, (u64*)d_m_out);
}

// ---------------------------------------------------------------------------------------
// Real and imaginary slot parts of complex-packed ciphertexts, each doubled:
//   re2 = ct + conj(ct),  im2 = -i (ct - conj(ct))   (-i = the monomial X^(N/2) applied three times, exact).
// ---------------------------------------------------------------------------------------
extern "C" int fesc_split_complex(fesc_ctx* ctx, const uint64_t* d_in, uint64_t* d_re2, uint64_t* d_im2, uint32_t batch,
                                  uint32_t n_limbs, uint32_t conj_key_id, void* stream) {
    if (!ctx || !d_in || !d_re2 || d_in == d_re2 || d_in == d_im2 || d_re2 == d_im2) return FESC_EINVAL;
    if (n_limbs == 0 || n_limbs > ctx->n_q) return fesc_fail(ctx, FESC_ELEVEL, "split_complex: level out of range");
    if (batch == 0) return FESC_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const uint32_t N = ctx->N;
    const size_t ctw = (size_t)2 * n_limbs * N;
    u64* scratch;
    int rc = ctx_scratch(ctx, ks_scratch_words(ctx, n_limbs, ks_chunk(ctx, batch)) * sizeof(u64), &scratch);
    if (rc != FESC_OK) return rc;
    const u64* in = (const u64*)d_in;
    u64 *re = (u64*)d_re2, *im = (u64*)d_im2;
    // conj(ct) into re, then im = ct - conj, re = ct + conj, im *= -i
    rc = rotate_internal(ctx, in, ctw, re, ctw, batch, n_limbs, conj_key_id, scratch, st, 0);
    if (rc != FESC_OK) return rc;
    const dim3 g((N + 255) / 256, 2 * n_limbs, batch);
    prof_begin(ctx, PF_POINTWISE, st);
    if (im) k_ct_addsub<<<g, 256, 0, st>>>(in, ctw, re, ctw, im, ctw, ctx->d_pc, N, n_limbs, 1);
    k_ct_addsub<<<g, 256, 0, st>>>(in, ctw, re, ctw, re, ctw, ctx->d_pc, N, n_limbs, 0);
    if (im) k_ct_mul_i<<<g, 256, 0, st>>>(im, ctw, im, ctw, ctx->d_pc, ctx->d_tw, N, n_limbs, 3);
    prof_end(ctx, PF_POINTWISE, st, im ? 3 : 1);
    FESC_CHECK_CUDA(ctx, cudaGetLastError());
    return FESC_OK;
}
