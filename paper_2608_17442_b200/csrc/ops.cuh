// Internal interfaces between the ciphertext-operation translation units.
#pragma once
#include "common.cuh"

// Scratch of one key-switch chunk (all [chunk][...][N] words):
//   dcoef [level]            the polynomial being switched, transformed to COEFF in place
//   ext   [beta][level+K]    converted digits; the rows of a digit's own limbs hold the polynomial itself (EVAL)
//   acc   [2][level+K]       inner-product accumulators
//   u     [2][level]         converted special-limb part
struct KsScratch {
    u64 *dcoef, *ext, *acc, *u;
};
size_t ks_scratch_words(const fesc_ctx* ctx, uint32_t level, uint32_t chunk);
KsScratch ks_scratch_carve(const fesc_ctx* ctx, u64* base, uint32_t level, uint32_t chunk);
uint32_t ks_chunk(const fesc_ctx* ctx, uint32_t batch);

int rotate_internal(fesc_ctx* ctx, const u64* in, size_t in_stride, u64* out, size_t out_stride, uint32_t batch,
                    uint32_t level, uint32_t key_id, u64* scratch, cudaStream_t st, int accumulate);
int rotate_hoisted_internal(fesc_ctx* ctx, const u64* in, size_t in_stride, u64* out, size_t out_stride,
                            size_t key_stride, uint32_t batch, uint32_t level, const uint32_t* key_ids, uint32_t n_keys,
                            u64* scratch, cudaStream_t st);
int rotate_sum_hoisted_internal(fesc_ctx* ctx, const u64* in, size_t in_stride, u64* out, size_t out_stride,
                                uint32_t batch, uint32_t level, const uint32_t* key_ids, uint32_t n_keys, u64* scratch,
                                cudaStream_t st);
int giant_sum_deferred_internal(fesc_ctx* ctx, u64* acc, uint32_t n_terms, size_t ct_words, uint32_t batch,
                                uint32_t level, uint32_t key_base, u64* scratch, cudaStream_t st);
int rescale_internal(fesc_ctx* ctx, const u64* in, size_t in_stride, u64* out, uint32_t batch, uint32_t level,
                     u64* scratch, cudaStream_t st);
int ctmul_internal(fesc_ctx* ctx, const u64* a, size_t a_stride, const u64* b, size_t b_stride, u64* out,
                   size_t out_stride, uint32_t batch, uint32_t level, u64* scratch, cudaStream_t st);
