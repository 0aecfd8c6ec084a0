// Rescale for callers that must not allocate device memory.
//
// Some hosts of this library cannot let a call reach cudaMalloc: code holding a fixed memory budget
// agreed with another allocator (a serving process that pre-partitions HBM), real-time loops where an
// allocation's implicit device synchronisation is not acceptable, plug-ins whose host forbids
// allocator calls on its threads.  fesc_rescale sizes its scratch from the context arena, which
// may grow on first use.  The entry point below does the same arithmetic with its scratch in a
// fixed device array that is part of the library image, so it never allocates.
#define FESC_DBG_FILE 9   // file id in the sites a debug build reports
#include "ops.cuh"

// Scratch of the rescale: the last limb of every polynomial of the batch (batch * 2 rows of N words),
// transformed in place to coefficient form.  4 MiB: 4 ciphertexts at N = 2^16, 64 at N = 2^12.
// Every GPU that loads the library holds this array until the process exits.
#define FESC_STATIC_SCRATCH_WORDS (4u * 2u * 65536u)
static __device__ __align__(256) unsigned long long g_rescale_scratch[FESC_STATIC_SCRATCH_WORDS];

// Device address of the array, looked up once per device ordinal.  The symbol's name is only a host-side
// handle; kernels need the address cudaGetSymbolAddress returns for the CURRENT device.  Under lazy module
// loading that lookup is what loads this module and places the array on the device, so the first call belongs
// at initialisation (it needs 4 MiB to be available).  The cache is written without locking: first calls on a
// device must not race across host threads; afterwards it is only read.
#define FESC_MAX_DEVICES 64
static u64* g_scratch_addr[FESC_MAX_DEVICES];

extern "C" int fesc_rescale_static(fesc_ctx* ctx, const uint64_t* d_in, uint64_t* d_out, uint32_t batch,
                                   uint32_t n_limbs, void* stream) {
    if (!ctx || !d_in || !d_out) return FESC_EINVAL;
    if (n_limbs < 2 || n_limbs > ctx->n_q) return fesc_fail(ctx, FESC_ELEVEL, "rescale_static: level out of range");
    if (batch == 0) return FESC_OK;
    if ((uint64_t)batch * 2 * ctx->N > FESC_STATIC_SCRATCH_WORDS)
        return fesc_fail(ctx, FESC_EINVAL,
                         "rescale_static: batch * 2 * N = " + std::to_string((uint64_t)batch * 2 * ctx->N) +
                             " words exceeds the static scratch of " + std::to_string(FESC_STATIC_SCRATCH_WORDS) +
                             " words; split the batch or use fesc_rescale");
    int dev = -1;
    FESC_CHECK_CUDA(ctx, cudaGetDevice(&dev));
    if (dev < 0 || dev >= FESC_MAX_DEVICES) return fesc_fail(ctx, FESC_EINVAL, "rescale_static: device index out of range");
    if (!g_scratch_addr[dev]) {   // first call on this device: do it before any stream capture starts
        void* p = nullptr;
        FESC_CHECK_CUDA(ctx, cudaGetSymbolAddress(&p, g_rescale_scratch));
        g_scratch_addr[dev] = (u64*)p;
        dbg_note_alloc(p, sizeof(g_rescale_scratch));      // a debug build checks the kernels' regions against known extents
    }
    return rescale_internal(ctx, (const u64*)d_in, (size_t)2 * n_limbs * ctx->N, (u64*)d_out, batch, n_limbs,
                            g_scratch_addr[dev], (cudaStream_t)stream);
}
