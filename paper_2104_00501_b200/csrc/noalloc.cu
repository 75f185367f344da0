// Ordered push that never allocates: the scratch of the sort-and-apply path lives in a
// fixed device array that is part of the library image.
#include <stdio.h>

#include "nups_internal.cuh"

// Scratch of nups_push_noalloc.  Every GPU that loads the library holds these bytes until
// the process exits.  Sized for NUPS_NOALLOC_MAX_ROWS rows: two key buffers, two index
// buffers, the radix histogram and its scan levels.
#define NUPS_NOALLOC_SCRATCH_BYTES (2u << 20)
static __device__ __align__(256) unsigned char g_noalloc_scratch[NUPS_NOALLOC_SCRATCH_BYTES];

// Device address of the array, looked up once per device.  In host code the array's name is
// only a stand-in for the symbol; a kernel must be given the address that the runtime
// returns for the device that is current.
#define NUPS_NOALLOC_MAX_DEVICES 64
static char* g_noalloc_addr[NUPS_NOALLOC_MAX_DEVICES];

extern "C" nups_status nups_push_noalloc(nups_store* s, const uint32_t* d_keys, uint64_t n, const void* d_delta_,
                                         void* stream)
{
    const float* d_delta = (const float*)d_delta_;
    if (!s || (n && (!d_keys || !d_delta))) return NUPS_EINVAL;
    if (!s->cfg.deterministic) return NUPS_ESTATE;
    if (n > NUPS_NOALLOC_MAX_ROWS) {
        snprintf(g_nups_cuda_err, sizeof(g_nups_cuda_err),
                 "nups_push_noalloc: %llu rows exceed the fixed scratch (at most %d rows per call)",
                 (unsigned long long)n, NUPS_NOALLOC_MAX_ROWS);
        return NUPS_EINVAL;
    }
    if (n == 0) return NUPS_OK;
    if (nups_push_scratch_bytes(s, n) > NUPS_NOALLOC_SCRATCH_BYTES) return NUPS_EINVAL;
    int dev = -1;
    CK(cudaGetDevice(&dev));
    if (dev != s->device || dev < 0 || dev >= NUPS_NOALLOC_MAX_DEVICES) return NUPS_ESTATE;
    if (!g_noalloc_addr[dev]) {
        void* p = nullptr;
        CK(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        g_noalloc_addr[dev] = (char*)p;
    }
    return nups_push_with_scratch(s, d_keys, n, 1, d_delta, nullptr, g_noalloc_addr[dev], (cudaStream_t)stream);
}
