// The CKKS steps around the NeRMS protocol (Alg. "one Block") on the projection packing
// idx(token, channel) = channel*T + token:
//   u  = y~ (.) y~                                   (the squares the protocol turns into an inverse RMS per token)
//   y^ = gamma_RMS (.) (y~ (.) br(s_RMS))            (the input of HEOutProj)
// br(s): the token factors sit in slots k < T of one ciphertext per token block; log2(n/T) rotate-right-and-add
// steps by T*2^b copy them to every channel of the block.  Products are relinearised and rescaled.
#define FESC_DBG_FILE 8   // file id in the sites a debug build reports
#include "ops.cuh"

// out[b] = ct[b] (.) pt[b] on both polynomials (pt_stride words between plaintexts)
// (out may be ct itself: every thread reads its words before it writes them)
__global__ void __launch_bounds__(256) k_ct_mul_pt(const u64* ct, size_t ct_stride, const u64* __restrict__ pt,
                                                   size_t pt_stride, u64* out, size_t out_stride,
                                                   const PrimeConst* __restrict__ pcs, uint32_t N, uint32_t level) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t l = blockIdx.y, b = blockIdx.z;
    if (c >= N) return;
    const PrimeConst pc = pcs[l];
    const size_t poly = (size_t)level * N, o = (size_t)l * N + c;
    if (!DBG_REGION(pt + (size_t)b * pt_stride + o - c, N * sizeof(u64))) return;
    for (int p = 0; p < 2; p++)
        if (!DBG_REGION(ct + (size_t)b * ct_stride + p * poly + o - c, N * sizeof(u64)) ||
            !DBG_REGION(out + (size_t)b * out_stride + p * poly + o - c, N * sizeof(u64)))
            return;
    const u64 w = pt[(size_t)b * pt_stride + o];
    out[(size_t)b * out_stride + o] = mulmod(ct[(size_t)b * ct_stride + o], w, pc);
    out[(size_t)b * out_stride + poly + o] = mulmod(ct[(size_t)b * ct_stride + poly + o], w, pc);
}

extern "C" int fesc_norm_square(fesc_ctx* ctx, const uint64_t* d_y, uint64_t* d_out, uint32_t batch, uint32_t n_limbs,
                                void* stream) {
    if (!ctx || !d_y || !d_out) return FESC_EINVAL;
    if (n_limbs < 2 || n_limbs > ctx->n_q) return fesc_fail(ctx, FESC_ELEVEL, "norm_square: level out of range");
    if (batch == 0) return FESC_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const uint32_t N = ctx->N, group = batch < 16 ? batch : 16;
    const size_t ctw = (size_t)2 * n_limbs * N, outw = (size_t)2 * (n_limbs - 1) * N;
    const size_t ks_words = ks_scratch_words(ctx, n_limbs, ks_chunk(ctx, group));
    const size_t rs_words = (size_t)group * 2 * N;
    u64* scratch;
    int rc = ctx_scratch(ctx, ((size_t)group * ctw + (ks_words > rs_words ? ks_words : rs_words)) * sizeof(u64), &scratch);
    if (rc != FESC_OK) return rc;
    u64* prod = scratch;
    u64* ks = scratch + (size_t)group * ctw;
    const u64* y = (const u64*)d_y;
    u64* out = (u64*)d_out;
    for (uint32_t b0 = 0; b0 < batch; b0 += group) {
        const uint32_t nb = batch - b0 < group ? batch - b0 : group;
        rc = ctmul_internal(ctx, y + (size_t)b0 * ctw, ctw, y + (size_t)b0 * ctw, ctw, prod, ctw, nb, n_limbs, ks, st);
        if (rc != FESC_OK) return rc;
        rc = rescale_internal(ctx, prod, ctw, out + (size_t)b0 * outw, nb, n_limbs, ks, st);
        if (rc != FESC_OK) return rc;
    }
    return FESC_OK;
}

extern "C" int fesc_norm_scale(fesc_ctx* ctx, const uint64_t* d_y, const uint64_t* d_s, const uint64_t* d_gamma,
                               const fesc_norm_desc* desc, uint64_t* d_out, void* stream) {
    if (!ctx || !d_y || !d_s || !d_gamma || !desc || !d_out) return FESC_EINVAL;
    const uint32_t T = desc->T, blocks = desc->blocks, tbs = desc->token_blocks, level = desc->n_limbs;
    const uint32_t N = ctx->N, n = N / 2;
    if (!blocks || !tbs) return fesc_fail(ctx, FESC_EINVAL, "norm_scale: empty dimension");
    if (!T || T > n || (T & (T - 1))) return fesc_fail(ctx, FESC_EINVAL, "norm_scale: T must be a power of two within the slots");
    if (level < 3 || level > ctx->n_q) return fesc_fail(ctx, FESC_ELEVEL, "norm_scale: level out of range");
    uint32_t steps = 0;
    while ((T << steps) < n) steps++;
    for (uint32_t b = 0; b < steps; b++)
        if (!ctx->keys.count(desc->key_base + b))
            return fesc_fail(ctx, FESC_ENOKEY, "norm_scale: missing Galois key " + std::to_string(desc->key_base + b));
    cudaStream_t st = (cudaStream_t)stream;
    const size_t ctw = (size_t)2 * level * N, ctw1 = (size_t)2 * (level - 1) * N, ctw2 = (size_t)2 * (level - 2) * N;
    const uint32_t widest = tbs > blocks ? tbs : blocks;
    const size_t ks_words = ks_scratch_words(ctx, level, ks_chunk(ctx, widest));
    const size_t rs_words = (size_t)widest * 2 * N;
    u64* scratch;
    int rc = ctx_scratch(ctx, ((size_t)2 * tbs * ctw + (size_t)blocks * (ctw + ctw1) + (ks_words > rs_words ? ks_words : rs_words)) *
                                  sizeof(u64), &scratch);
    if (rc != FESC_OK) return rc;
    u64* f[2] = {scratch, scratch + (size_t)tbs * ctw};      // br(s) of every token block, ping-pong
    u64* prod = scratch + (size_t)2 * tbs * ctw;              // [blocks] at `level`
    u64* prod1 = prod + (size_t)blocks * ctw;                 // [blocks] at level-1
    u64* ks = prod1 + (size_t)blocks * ctw1;
    FESC_CHECK_CUDA(ctx, cudaMemcpyAsync(f[0], d_s, (size_t)tbs * ctw * sizeof(u64), cudaMemcpyDeviceToDevice, st));
    uint32_t cur = 0;
    for (uint32_t b = 0; b < steps; b++) {                    // f += rot(f, -(T << b)), all token blocks at once
        FESC_CHECK_CUDA(ctx, cudaMemcpyAsync(f[cur ^ 1], f[cur], (size_t)tbs * ctw * sizeof(u64), cudaMemcpyDeviceToDevice, st));
        rc = rotate_internal(ctx, f[cur], ctw, f[cur ^ 1], ctw, tbs, level, desc->key_base + b, ks, st, 1);
        if (rc != FESC_OK) return rc;
        cur ^= 1;
    }
    const u64* y = (const u64*)d_y;
    u64* out = (u64*)d_out;
    const dim3 grid((N + 255) / 256, level - 1, blocks);
    for (uint32_t tb = 0; tb < tbs; tb++) {
        rc = ctmul_internal(ctx, y + (size_t)tb * blocks * ctw, ctw, f[cur] + (size_t)tb * ctw, 0, prod, ctw, blocks, level, ks, st);
        if (rc != FESC_OK) return rc;
        if ((rc = rescale_internal(ctx, prod, ctw, prod1, blocks, level, ks, st)) != FESC_OK) return rc;
        prof_begin(ctx, PF_POINTWISE, st);
        k_ct_mul_pt<<<grid, 256, 0, st>>>(prod1, ctw1, (const u64*)d_gamma, (size_t)(level - 1) * N, prod1, ctw1, ctx->d_pc, N, level - 1);
        prof_end(ctx, PF_POINTWISE, st);
        FESC_CHECK_CUDA(ctx, cudaGetLastError());
        rc = rescale_internal(ctx, prod1, ctw1, out + (size_t)tb * blocks * ctw2, blocks, level - 1, ks, st);
        if (rc != FESC_OK) return rc;
    }
    return FESC_OK;
}
