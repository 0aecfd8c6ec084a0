// Causal depthwise convolution on the projection packing (Sec. "Causal Depthwise Convolution", Eq. conv1d_depthwise):
//   eta = b + sum_r M_r (.) rho(q; delta_r),   slot idx(token, channel) = channel*T + token.
// Tap r >= 1 of token k reads token k-r: inside a token block that is rho(q; -r) masked to tokens k >= r (M_r); the
// first r tokens of a block read the previous block's last tokens, rho(q_prev; T - r) masked to k < r (M'_r).
// Every ciphertext is decomposed once and rotated by its 2(d_conv-1) amounts (hoisted rotations); the rotations by
// T - r are kept for the next token block.  The masked sums use the plain ct-pt multiply-accumulate, then the bias
// plaintext is added to c0 and the block is rescaled.
#define FESC_DBG_FILE 7   // file id in the sites a debug build reports
#include "ops.cuh"

// c0 of every ciphertext += its plaintext (pt_stride words between plaintexts)
__global__ void __launch_bounds__(256) k_ct_add_pt(u64* __restrict__ ct, size_t ct_stride, const u64* __restrict__ pt,
                                                   size_t pt_stride, const PrimeConst* __restrict__ pcs, uint32_t N) {
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t l = blockIdx.y, b = blockIdx.z;
    if (c >= N) return;
    u64* o = ct + (size_t)b * ct_stride + (size_t)l * N + c;
    if (!DBG_REGION(o - c, N * sizeof(u64)) || !DBG_REGION(pt + (size_t)b * pt_stride + (size_t)l * N, N * sizeof(u64))) return;
    *o = addmod(*o, pt[(size_t)b * pt_stride + (size_t)l * N + c], pcs[l].q);
}

extern "C" int fesc_conv(fesc_ctx* ctx, const uint64_t* d_ct_in, const uint64_t* d_masks, const uint64_t* d_bias,
                         const fesc_conv_desc* desc, uint64_t* d_ct_out, void* stream) {
    if (!ctx || !d_ct_in || !d_masks || !d_bias || !desc || !d_ct_out) return FESC_EINVAL;
    const uint32_t d = desc->d_conv, T = desc->T, blocks = desc->blocks, tbs = desc->token_blocks, level = desc->n_limbs;
    const uint32_t N = ctx->N;
    if (!d || d > 8 || !blocks || !tbs) return fesc_fail(ctx, FESC_EINVAL, "conv: empty dimension or more than 8 taps");
    if (!T || (N / 2) % T || d > T) return fesc_fail(ctx, FESC_EINVAL, "conv: T must divide the slot count and exceed the taps");
    if (level < 2 || level > ctx->n_q) return fesc_fail(ctx, FESC_ELEVEL, "conv: level out of range");
    const uint32_t taps = d - 1;
    std::vector<uint32_t> ids;
    for (uint32_t r = 1; r < d; r++) ids.push_back(desc->key_base + r);            // rotation by -r
    for (uint32_t r = 1; r < d; r++) ids.push_back(desc->key_base + d + r);        // rotation by T - r
    for (uint32_t i = 0; i < ids.size(); i++)
        if ((i < taps || tbs > 1) && !ctx->keys.count(ids[i]))
            return fesc_fail(ctx, FESC_ENOKEY, "conv: missing Galois key " + std::to_string(ids[i]));
    cudaStream_t st = (cudaStream_t)stream;
    const size_t ctw = (size_t)2 * level * N, ptw = (size_t)level * N;
    const size_t rot_words = (size_t)2 * taps * blocks * ctw;       // one buffer: [2*taps][blocks] ciphertexts
    const size_t ks_words = ks_scratch_words(ctx, level, ks_chunk(ctx, blocks));
    const size_t rs_words = (size_t)blocks * 2 * N;
    u64* scratch;
    int rc = ctx_scratch(ctx, (2 * rot_words + (size_t)blocks * ctw + (ks_words > rs_words ? ks_words : rs_words)) * sizeof(u64),
                         &scratch);
    if (rc != FESC_OK) return rc;
    u64* rot[2] = {scratch, scratch + rot_words};
    u64* acc = scratch + 2 * rot_words;
    u64* ks = acc + (size_t)blocks * ctw;
    const u64* in = (const u64*)d_ct_in;
    const u64* masks = (const u64*)d_masks;
    const size_t mask_stride = (size_t)(2 * d - 1) * ptw;
    u64* out = (u64*)d_ct_out;
    for (uint32_t tb = 0; tb < tbs; tb++) {
        const u64* cur = in + (size_t)tb * blocks * ctw;
        u64* R = rot[tb & 1];
        const u64* Rprev = rot[(tb & 1) ^ 1];
        const uint32_t n_keys = taps ? (tb + 1 < tbs ? 2 * taps : taps) : 0;
        if (n_keys) {
            rc = rotate_hoisted_internal(ctx, cur, ctw, R, ctw, (size_t)blocks * ctw, blocks, level, ids.data(), n_keys, ks, st);
            if (rc != FESC_OK) return rc;
        }
        FESC_CHECK_CUDA(ctx, cudaMemsetAsync(acc, 0, (size_t)blocks * ctw * sizeof(u64), st));
        auto mac = [&](const u64* ct, const u64* pt) {
            return fesc_ct_pt_mac(ctx, (const uint64_t*)ct, (const uint64_t*)pt, mask_stride, (uint64_t*)acc, blocks, level, stream);
        };
        if ((rc = mac(cur, masks)) != FESC_OK) return rc;
        for (uint32_t r = 1; r < d; r++) {
            if ((rc = mac(R + (size_t)(r - 1) * blocks * ctw, masks + (size_t)r * ptw)) != FESC_OK) return rc;
            if (tb > 0) {
                rc = mac(Rprev + (size_t)(taps + r - 1) * blocks * ctw, masks + (size_t)(d - 1 + r) * ptw);
                if (rc != FESC_OK) return rc;
            }
        }
        prof_begin(ctx, PF_POINTWISE, st);
        k_ct_add_pt<<<dim3((N + 255) / 256, level, blocks), 256, 0, st>>>(acc, ctw, (const u64*)d_bias, ptw, ctx->d_pc, N);
        prof_end(ctx, PF_POINTWISE, st);
        FESC_CHECK_CUDA(ctx, cudaGetLastError());
        rc = rescale_internal(ctx, acc, ctw, out + (size_t)tb * blocks * 2 * (level - 1) * N, blocks, level, ks, st);
        if (rc != FESC_OK) return rc;
    }
    return FESC_OK;
}
