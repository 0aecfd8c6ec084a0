// BSGS accumulate on the tensor cores with operands stored as byte-plane fragments.
//
// For one coefficient c of one limb the giant-step accumulators of a projection (App. "Projection Kernel Breakdown",
// acc_p = sum_{g,q} rot(x^(g), qT) (.) D_{g,p,q}) are a small dense integer matrix product over the terms t = (g,q):
//   S[(tb,pol)][bp] = sum_t x_t[(tb,pol)] * w_t[bp].
// Every residue below 2^56 is cut into 7 bytes; with D[k][j] = sum_t w_t.byte(k) * x_t.byte(j) (exact s32 sums of
// mma.sync m16n8k32 u8 x u8)  S = sum_{k,j} 256^(k+j) D[k][j].
//
// The plaintext diagonals are weights: they are packed ONCE (fesc_linear_pack_diags) into the exact register
// fragments of the instruction, tile by tile, so that a CTA streams ONE contiguous run of bytes per (b,p) tile with
// bulk asynchronous copies and a warp fetches a whole 16 x 32 operand tile with one 16-byte shared-memory load per
// lane: no byte shuffling, no bank conflicts and no address arithmetic in the inner loop.  The rotated inputs of a
// group of token blocks are packed the same way by a small kernel before the accumulate (their fragments then live
// in registers for the whole CTA when there are at most 96 terms).
//
// Packed layout.  A "fragment image" is the operand of one coefficient for one k-step (32 terms) and one tile of
// 8 rows (8 (b,p) outputs on the diagonal side, 4 token blocks x 2 polynomials on the input side), 1792 bytes:
//   diagonal side: m-tile m = 0..2 holds byte planes (2m, 2m+1): [lane 32][a0 a1 a2 a3] (512 bytes each), m-tile 3
//                  holds plane 6: [lane 32][a0 a2] (256 bytes); lane = 4 g + tg reads row g (output g of the tile),
//                  a0/a1 = planes 2m / 2m+1 of terms 4tg..4tg+3, a2/a3 the same planes of terms 16+4tg..16+4tg+3;
//   input side:    n-tile j = 0..6 holds plane j: [lane 32][b0 b1] (256 bytes each); lane = 4 g + tg reads column g
//                  ((token block, polynomial) g of the tile), b0 = terms 4tg..4tg+3, b1 = terms 16+4tg..16+4tg+3.
// Images are ordered [row tile][limb][coefficient tile of 8][k-step][coefficient 8], so the 8 x ksteps images one
// CTA needs for one (b,p) tile are contiguous.  Rows and terms beyond the valid ones are zero.
#define FESC_DBG_FILE 5   // file id in the sites a debug build reports
#include "ops.cuh"

#define PK_CW 8
#define PK_FRAG 1792
#define PK_STAGE (PK_CW * PK_FRAG)
#define PK_STAGES 7
#define PK_ROWP 9
#define PK_BLK (32 * PK_ROWP + 1)

size_t bsgs_packed_bytes(uint32_t N, uint32_t level, uint32_t rows, uint32_t terms) {
    const size_t row_tiles = (rows + 7) / 8, ksteps = (terms + 31) / 32;
    return row_tiles * level * (size_t)N * ksteps * PK_FRAG;
}

// One CTA packs one (row tile, limb, coefficient tile, k-step): 8 rows x 32 terms x 8 coefficients in, 8 images out.
// Row r of the source: diagonal side  src + r * stride_hi;  input side  src + (r >> 1) * stride_hi + (r & 1) * stride_lo.
template <bool A_SIDE>
__global__ void __launch_bounds__(256) k_pack_fragments(const u64* __restrict__ src, uint8_t* __restrict__ dst, uint32_t N,
                                                        uint32_t level, uint32_t rows, uint32_t terms, uint32_t ksteps,
                                                        size_t stride_hi, size_t stride_lo, size_t term_stride) {
    __shared__ u64 sm[8 * PK_BLK];
    const uint32_t tid = threadIdx.x, cw = tid & 7, rw = tid >> 3;
    const uint32_t ct = blockIdx.x, l = blockIdx.y, tile = blockIdx.z / ksteps, ks = blockIdx.z - tile * ksteps;
    const uint32_t t = (ks << 5) + rw;
#ifdef FESC_DEBUG_BOUNDS
    {   // the same outcome for every thread of the CTA (there is a barrier below): all 8 rows x 32 terms, one limb row each
        bool ok = DBG_REGION(dst + ((((size_t)tile * level + l) * gridDim.x + ct) * ksteps + ks) * PK_STAGE, PK_STAGE);
        for (uint32_t g = 0; g < 8 && ok; g++)
            for (uint32_t tt = ks << 5; tt < (ks << 5) + 32 && tt < terms && ok; tt++) {
                const uint32_t r = tile * 8 + g;
                if (r >= rows) break;
                const size_t off = A_SIDE ? (size_t)r * stride_hi : (size_t)(r >> 1) * stride_hi + (size_t)(r & 1) * stride_lo;
                ok = DBG_REGION(src + off + (size_t)tt * term_stride + (size_t)l * N + ct * PK_CW, PK_CW * sizeof(u64));
            }
        if (!ok) return;
    }
#endif
#pragma unroll
    for (uint32_t g = 0; g < 8; g++) {
        const uint32_t r = tile * 8 + g;
        u64 v = 0;
        if (r < rows && t < terms) {
            const size_t off = A_SIDE ? (size_t)r * stride_hi : (size_t)(r >> 1) * stride_hi + (size_t)(r & 1) * stride_lo;
            v = src[off + (size_t)t * term_stride + (size_t)l * N + ct * PK_CW + cw];
        }
        sm[g * PK_BLK + rw * PK_ROWP + cw] = v;
    }
    __syncthreads();
    const uint32_t warp = tid >> 5, lane = tid & 31, g = lane >> 2, tg = lane & 3;
    const u64* p = sm + g * PK_BLK + (4 * tg) * PK_ROWP + warp;
    uint32_t lo[7], hi[7];
    byte_planes4(p[0], p[PK_ROWP], p[2 * PK_ROWP], p[3 * PK_ROWP], lo);
    byte_planes4(p[16 * PK_ROWP], p[17 * PK_ROWP], p[18 * PK_ROWP], p[19 * PK_ROWP], hi);
    uint8_t* out = dst + ((((size_t)tile * level + l) * gridDim.x + ct) * ksteps + ks) * PK_STAGE + warp * PK_FRAG;
    if (A_SIDE) {
#pragma unroll
        for (int m = 0; m < 3; m++)
            *(uint4*)(out + m * 512 + lane * 16) = make_uint4(lo[2 * m], lo[2 * m + 1], hi[2 * m], hi[2 * m + 1]);
        *(uint2*)(out + 1536 + lane * 8) = make_uint2(lo[6], hi[6]);
    } else {
#pragma unroll
        for (int j = 0; j < 7; j++) *(uint2*)(out + j * 256 + lane * 8) = make_uint2(lo[j], hi[j]);
    }
}

int bsgs_pack_inputs(fesc_ctx* ctx, const u64* rot, uint8_t* xpk, uint32_t level, uint32_t tbs, uint32_t terms,
                     cudaStream_t st) {
    const uint32_t N = ctx->N, ksteps = (terms + 31) / 32, tiles = (2 * tbs + 7) / 8;
    const size_t poly = (size_t)level * N, ctw = 2 * poly;
    dim3 grid(N / PK_CW, level, tiles * ksteps);
    if (grid.z > 65535 || level > 65535) return fesc_fail(ctx, FESC_EINVAL, "linear: too many packing tiles");
    prof_begin(ctx, PF_POINTWISE, st);
    k_pack_fragments<false><<<grid, 256, 0, st>>>(rot, xpk, N, level, 2 * tbs, terms, ksteps, (size_t)terms * ctw, poly, ctw);
    prof_end(ctx, PF_POINTWISE, st);
    FESC_CHECK_CUDA(ctx, cudaGetLastError());
    return FESC_OK;
}

// Accumulate: CTA = (half a coefficient tile, limb, tile of 4 token blocks) = 4 warps, one coefficient each; three
// CTAs share an SM, so every scheduler holds three warps: while one recombines its finished tile (a latency-bound
// chain of integer and FP64 operations) the other two keep the tensor pipe busy.  Every warp streams the diagonal
// images of ITS coefficient (1792 bytes per k-step, one bulk asynchronous copy each) through a private ring of
// PK_STAGES slots, each slot with its own barrier: the warp that consumed a slot requests the copy that refills it,
// so warps never wait for one another.  The input fragments of the coefficient (at most 6 k-steps, ring and inputs together at most 10 slots) are copied once
// into shared memory the same way.  Every barrier wait is bounded; a wait that runs out sets the status word (3), the
// warp waits (bounded) for its other copies in flight and leaves.
#define PK_WARPS 4
template <bool FP, int KSR, int ST>
__global__ void __launch_bounds__(32 * PK_WARPS, 3) k_bsgs_accumulate_packed(
    const uint8_t* __restrict__ xpk, const uint8_t* __restrict__ dpk, u64* __restrict__ acc,
    const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level, uint32_t tbs, uint32_t ksteps, uint32_t bp_count,
    uint32_t dshift, uint32_t* __restrict__ status) {
    // per warp: ST ring slots, KSR input images; then per warp ST + 1 barriers
    extern __shared__ __align__(128) uint8_t ring[];
    constexpr uint32_t WARP_BYTES = (ST + KSR) * PK_FRAG;
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tg = lane & 3;
    // blockIdx.x = (coefficient half-tile) * token-block tiles + token-block tile: the CTAs that stream the same images
    // for different token blocks start together, so only the first of them reads the images from HBM
    const uint32_t tbts = (tbs + 3) >> 2, tbt = blockIdx.x % tbts, half_tile = blockIdx.x / tbts;
    const uint32_t ct = half_tile >> 1, coef = (half_tile & 1) * PK_WARPS + warp, l = blockIdx.y;
    const uint32_t tiles = gridDim.x / (2 * tbts);
    const uint32_t bp_tiles = (bp_count + 7) >> 3, total = bp_tiles * ksteps;
    const uint32_t my_ring = (uint32_t)__cvta_generic_to_shared(ring) + warp * WARP_BYTES;
    const uint32_t my_bar = (uint32_t)__cvta_generic_to_shared(ring) + PK_WARPS * WARP_BYTES + warp * ((ST + 1) * 8);
    const uint8_t* my_img = ring + warp * WARP_BYTES;
    // images of this warp's coefficient: k-steps of one (b,p) tile are PK_STAGE apart, tiles tile_stride apart.  Periodic
    // diagonals (dshift > 0) hold one image per aligned run of 2^dshift coefficients: the image of a ring 2^dshift times
    // smaller, shared by the coefficients of the run.
    const uint32_t run = (ct * PK_CW + coef) >> dshift, tiles_d = tiles >> dshift;
    const uint8_t* src = dpk + ((size_t)l * tiles_d + (run >> 3)) * ksteps * PK_STAGE + (run & 7) * PK_FRAG;
    const size_t tile_stride = (size_t)level * tiles_d * ksteps * PK_STAGE;
    const uint8_t* ximg = xpk + ((((size_t)tbt * level + l) * tiles + ct) * ksteps * PK_CW + coef) * PK_FRAG;
#ifdef FESC_DEBUG_BOUNDS
    {   // the same outcome for every thread of the CTA (barriers follow): the streams of all four warps and the output rows
        bool ok = true;
        for (uint32_t w = 0; w < PK_WARPS && ok; w++) {
            const uint32_t cf = (half_tile & 1) * PK_WARPS + w, rn = (ct * PK_CW + cf) >> dshift;
            const uint8_t* sw = dpk + ((size_t)l * tiles_d + (rn >> 3)) * ksteps * PK_STAGE + (rn & 7) * PK_FRAG;
            for (uint32_t bt = 0; bt < bp_tiles && ok; bt++)
                ok = DBG_REGION(sw + bt * tile_stride, (size_t)(ksteps - 1) * PK_STAGE + PK_FRAG);
            ok = ok && DBG_REGION(xpk + ((((size_t)tbt * level + l) * tiles + ct) * ksteps * PK_CW + cf) * PK_FRAG,
                                  (size_t)(ksteps - 1) * PK_STAGE + PK_FRAG);
        }
        for (uint32_t tb = tbt * 4; tb < tbt * 4 + 4 && tb < tbs && ok; tb++)
            ok = DBG_REGION(acc + (size_t)tb * bp_count * 2 * level * N, (size_t)bp_count * 2 * level * N * sizeof(u64));
        if (!ok) return;
    }
#endif
    uint32_t ld_ks = 0, ld_s = 0;                         // next stage to request (lane 0)
    auto request = [&](uint32_t slot) {
        mbar_expect_tx(my_bar + slot * 8, PK_FRAG);
        bulk_g2s(my_ring + slot * PK_FRAG, src + (size_t)ld_ks * PK_STAGE, PK_FRAG, my_bar + slot * 8);
        if (++ld_ks == ksteps) ld_ks = 0, src += tile_stride;
        ld_s++;
    };
    if (lane == 0) {
        for (uint32_t i = 0; i <= ST; i++) mbar_init(my_bar + i * 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (KSR > 0) {
            mbar_expect_tx(my_bar + ST * 8, KSR * PK_FRAG);
            for (uint32_t k = 0; k < KSR; k++)
                bulk_g2s(my_ring + (ST + k) * PK_FRAG, ximg + (size_t)k * PK_STAGE, PK_FRAG, my_bar + ST * 8);
        }
        for (uint32_t i = 0; i < ST && i < total; i++) request(i);
    }
    __syncwarp();
    const PrimeConst pc = pcs[l];
    const size_t poly = (size_t)level * N, ctw = 2 * poly;
    double c32 = 0, c64 = 0, c96 = 0;
    if (FP) {
        c32 = fp_reduce(4294967296.0, pc.qd, pc.qinvd);
        c64 = fp_modmul(c32, c32, pc.qd, pc.qinvd);
        c96 = fp_modmul(c64, c32, pc.qd, pc.qinvd);
    }
    const uint32_t out_bar = (uint32_t)__cvta_generic_to_shared(ring) + PK_WARPS * (WARP_BYTES + (ST + 1) * 8) + 2 * 256 * 8;
    if (tid == 0) {
        mbar_init(out_bar, PK_WARPS);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    int d[4][7][4];
    int z0 = 0, z1 = 0, z2 = 0, z3 = 0;                   // a fixed quad of zero addends (see imma_u8_zero)
    asm volatile("" : "+r"(z0), "+r"(z1), "+r"(z2), "+r"(z3));
    uint32_t slot = 0, phase = 0, s = 0;
    bool ok = KSR == 0 || !mbar_wait_bounded(my_bar + ST * 8, 0);
    const bool x_ok = ok;
    auto mma_stage = [&](const uint8_t* xfrag, bool first) {
        if (mbar_wait_bounded(my_bar + slot * 8, phase)) {
            ok = false;
            return;
        }
        const uint8_t* img = my_img + slot * PK_FRAG;
        const uint4 a0 = *(const uint4*)(img + lane * 16), a1 = *(const uint4*)(img + 512 + lane * 16);
        const uint4 a2 = *(const uint4*)(img + 1024 + lane * 16);
        uint4 a3;                                              // plane 6 and an empty plane
        a3.x = *(const uint32_t*)(img + 1536 + lane * 8);
        a3.z = *(const uint32_t*)(img + 1540 + lane * 8);
        a3.y = a3.w = 0u;
#pragma unroll
        for (int j = 0; j < 7; j++) {
            const uint2 b = KSR > 0 ? *(const uint2*)(xfrag + j * 256 + lane * 8)
                                    : __ldg((const uint2*)(xfrag + j * 256 + lane * 8));
            if (first) {
                imma_u8_zero(d[0][j], a0.x, a0.y, a0.z, a0.w, b.x, b.y, z0, z1, z2, z3);
                imma_u8_zero(d[1][j], a1.x, a1.y, a1.z, a1.w, b.x, b.y, z0, z1, z2, z3);
                imma_u8_zero(d[2][j], a2.x, a2.y, a2.z, a2.w, b.x, b.y, z0, z1, z2, z3);
                imma_u8_zero(d[3][j], a3.x, a3.y, a3.z, a3.w, b.x, b.y, z0, z1, z2, z3);
            } else {
                imma_u8(d[0][j], a0.x, a0.y, a0.z, a0.w, b.x, b.y);
                imma_u8(d[1][j], a1.x, a1.y, a1.z, a1.w, b.x, b.y);
                imma_u8(d[2][j], a2.x, a2.y, a2.z, a2.w, b.x, b.y);
                imma_u8(d[3][j], a3.x, a3.y, a3.z, a3.w, b.x, b.y);
            }
        }
        // The products above consumed every loaded register of every lane, so all reads of the slot have returned and
        // the slot can take its next image (a read that has completed cannot be affected by a later asynchronous
        // write, so no proxy fence is needed on this write-after-read path).
        __syncwarp();
        if (lane == 0 && ld_s < total) request(slot);
        s++;
        if (++slot == ST) slot = 0, phase ^= 1;
    };
#pragma unroll 1
    for (uint32_t bt = 0; bt < bp_tiles && ok; bt++) {
        if (KSR > 0) {
#pragma unroll
            for (int k = 0; k < (KSR > 0 ? KSR : 1); k++)
                if (ok) mma_stage(my_img + (ST + k) * PK_FRAG, k == 0);
        } else {
#pragma unroll 1
            for (uint32_t k = 0; k < ksteps && ok; k++) mma_stage(ximg + (size_t)k * PK_STAGE, k == 0);
        }
        if (!ok) break;
        // lane (g, tg) holds output bp = 8 bt + g of token block 4 tbt + tg, both polynomials.  The four warps of the
        // CTA (four neighbouring coefficients) exchange their results through shared memory so that every output row
        // receives one full 32-byte sector instead of four separate words.
        u64* stage_out = (u64*)(ring + PK_WARPS * (WARP_BYTES + (ST + 1) * 8)) + (bt & 1) * 256;
        stage_out[(lane * 2) * PK_WARPS + warp] = imma_recombine<FP>(d, 0, pc, c32, c64, c96);
        stage_out[(lane * 2 + 1) * PK_WARPS + warp] = imma_recombine<FP>(d, 1, pc, c32, c64, c96);
        // CTA-wide hand-over on a shared-memory barrier (one arrival per warp) so that this wait is bounded too
        __syncwarp();
        if (lane == 0) mbar_arrive(out_bar);
        if (mbar_wait_bounded(out_bar, bt & 1)) {
            ok = false;
            break;
        }
        {
            const uint32_t row = tid >> 1, rl = row >> 1, rg = rl >> 2, rtg = rl & 3;     // row = (lane of the owner) * 2 + polynomial
            const uint32_t bp = bt * 8 + rg, tb = tbt * 4 + rtg;
            if (bp < bp_count && tb < tbs) {
                const ulonglong2 v = *(const ulonglong2*)(stage_out + row * PK_WARPS + (tid & 1) * 2);
                u64* dst = acc + ((size_t)tb * bp_count + bp) * ctw + (row & 1) * poly + (size_t)l * N + ct * PK_CW +
                           (half_tile & 1) * PK_WARPS + (tid & 1) * 2;
                *(ulonglong2*)dst = v;
            }
        }
    }
    if (!ok) {
        // A copy never arrived.  The copies requested after the missing stage may still be in flight: give each a
        // bounded wait before this CTA's shared memory can be handed on.
        if (lane == 0) {
            atomicExch(status, 3u);
            for (uint32_t sp = x_ok ? s + 1 : 0; sp < ld_s; sp++)
                mbar_wait_bounded(my_bar + (sp % ST) * 8, (sp / ST) & 1);
        }
        __syncwarp();
    }
}

int bsgs_accumulate_packed(fesc_ctx* ctx, const uint8_t* xpk, const uint8_t* dpk, u64* acc, uint32_t level, uint32_t tbs,
                           uint32_t terms, uint32_t bp_count, bool fp, uint32_t dshift, cudaStream_t st) {
    const uint32_t N = ctx->N, ksteps = (terms + 31) / 32;
    dim3 grid(2 * (N / PK_CW) * ((tbs + 3) / 4), level);
#define PK_LAUNCH(FP, KSR, ST)                                                                                    \
    do {                                                                                                          \
        const size_t smem = (size_t)PK_WARPS * ((ST + KSR) * PK_FRAG + (ST + 1) * 8) + 2 * 256 * 8 + 8;           \
        auto kern = k_bsgs_accumulate_packed<FP, KSR, ST>;                                                        \
        FESC_CHECK_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        kern<<<grid, 32 * PK_WARPS, smem, st>>>(xpk, dpk, acc, ctx->d_pc, N, level, tbs, ksteps, bp_count, dshift, \
                                                ctx->d_status);                                                   \
    } while (0)
    // input fragments of up to 6 k-steps stay in shared memory (ring + inputs = 10 slots per warp, so that three CTAs
    // still share an SM); longer sums read them through L1 / L2 at every step
#define PK_PICK(FP)                                   \
    do {                                              \
        if (ksteps == 1) PK_LAUNCH(FP, 1, PK_STAGES); \
        else if (ksteps == 2) PK_LAUNCH(FP, 2, PK_STAGES); \
        else if (ksteps == 3) PK_LAUNCH(FP, 3, PK_STAGES); \
        else if (ksteps == 4) PK_LAUNCH(FP, 4, 6);    \
        else if (ksteps == 5) PK_LAUNCH(FP, 5, 5);    \
        else if (ksteps == 6) PK_LAUNCH(FP, 6, 4);    \
        else PK_LAUNCH(FP, 0, PK_STAGES);             \
    } while (0)
    prof_begin(ctx, PF_BSGS, st);
    if (fp) PK_PICK(true);
    else PK_PICK(false);
#undef PK_PICK
#undef PK_LAUNCH
    prof_end(ctx, PF_BSGS, st);
    FESC_CHECK_CUDA(ctx, cudaGetLastError());
    return FESC_OK;
}

static uint32_t max_prime_bits(const fesc_ctx* ctx, uint32_t level) {
    uint32_t qbits = 0;
    for (uint32_t i = 0; i < level; i++) {
        const uint32_t b = 64 - __builtin_clzll(ctx->q[i]);
        if (b > qbits) qbits = b;
    }
    return qbits;
}
bool bsgs_packed_supported(const fesc_ctx* ctx, uint32_t level, uint32_t terms, uint32_t dshift) {
    return ctx->N % PK_CW == 0 && level >= 1 && level <= ctx->n_q && max_prime_bits(ctx, level) <= 56 && terms >= 1 &&
           terms <= 512 && dshift < 32 && (ctx->N >> dshift) >= PK_CW;
}

extern "C" size_t fesc_linear_packed_bytes(const fesc_ctx* ctx, const fesc_bsgs_desc* desc) {
    if (!ctx || !desc) return 0;
    if (desc->diag_run_log2 >= 32) return 0;
    return bsgs_packed_bytes(ctx->N >> desc->diag_run_log2, desc->n_limbs, desc->out_blocks * desc->n2, desc->in_blocks * desc->n1);
}

extern "C" int fesc_linear_pack_diags(fesc_ctx* ctx, const uint64_t* d_diags, const fesc_bsgs_desc* desc, uint32_t first,
                                      uint32_t count, void* d_packed, void* stream) {
    if (!ctx || !d_diags || !desc || !d_packed) return FESC_EINVAL;
    const uint32_t level = desc->n_limbs, terms = desc->in_blocks * desc->n1, bp_count = desc->out_blocks * desc->n2;
    if (!bsgs_packed_supported(ctx, level, terms, desc->diag_run_log2))
        return fesc_fail(ctx, FESC_EINVAL, "pack_diags: needs N a multiple of 8, primes below 2^56, at most 512 terms and runs that leave 8 words per limb");
    const uint32_t N = ctx->N >> desc->diag_run_log2;       // words per limb of the diagonals handed in
    if (first % 8 || first >= bp_count || !count || count > bp_count - first)
        return fesc_fail(ctx, FESC_EINVAL, "pack_diags: the range must start at a multiple of 8 and lie inside the (b,p) pairs");
    if ((first + count) % 8 && first + count != bp_count)
        return fesc_fail(ctx, FESC_EINVAL, "pack_diags: only the last range may end inside a tile of 8");
    const uint32_t ksteps = (terms + 31) / 32, tiles = (count + 7) / 8;
    const size_t poly = (size_t)level * N;
    dim3 grid(N / PK_CW, level, tiles * ksteps);
    if (grid.z > 65535 || level > 65535) return fesc_fail(ctx, FESC_EINVAL, "pack_diags: range too large for one call");
    uint8_t* dst = (uint8_t*)d_packed + (size_t)(first / 8) * level * N * ksteps * PK_FRAG;
    k_pack_fragments<true><<<grid, 256, 0, (cudaStream_t)stream>>>((const u64*)d_diags, dst, N, level, count, terms, ksteps,
                                                                   (size_t)terms * poly, 0, poly);
    ctx->counters[4] += 1;
    FESC_CHECK_CUDA(ctx, cudaGetLastError());
    return FESC_OK;
}
