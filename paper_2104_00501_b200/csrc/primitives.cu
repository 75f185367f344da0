// Device-wide building blocks used off the hot path (hot-set selection, alias build,
// ordered push): exclusive prefix sum over uint64 and a stable LSD radix sort of
// (uint64 key, uint32 value) pairs.
#include "nups_internal.cuh"

namespace {

constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = 8;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;   // 2048 values per block

__device__ __forceinline__ unsigned long long block_exclusive_scan(unsigned long long x, unsigned long long* total,
                                                                   unsigned long long* sh /* [33] */)
{
    // exclusive scan of one value per thread over a 256-thread block
    unsigned lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long inc = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= (unsigned)o) inc += y;
    }
    if (lane == 31) sh[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        unsigned long long w = lane < (SCAN_THREADS / 32) ? sh[lane] : 0ull;
        unsigned long long winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, winc, o);
            if (lane >= (unsigned)o) winc += y;
        }
        if (lane < (SCAN_THREADS / 32)) sh[lane] = winc - w;
        if (lane == (SCAN_THREADS / 32) - 1) sh[32] = winc;
    }
    __syncthreads();
    unsigned long long res = sh[warp] + inc - x;
    *total = sh[32];
    __syncthreads();
    return res;
}

__global__ void scan_block_sums(const unsigned long long* __restrict__ in, unsigned long long* __restrict__ bsum,
                                uint64_t n)
{
    __shared__ unsigned long long sh[33];
    uint64_t base = (uint64_t)blockIdx.x * SCAN_TILE + (uint64_t)threadIdx.x * SCAN_ITEMS;
    unsigned long long t = 0;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i)
        if (base + i < n) t += in[base + i];
    unsigned long long total;
    block_exclusive_scan(t, &total, sh);
    if (threadIdx.x == 0) bsum[blockIdx.x] = total;
}

// one block scans up to SCAN_TILE values in place
__global__ void scan_single_block(unsigned long long* data, uint64_t n, unsigned long long* total_out)
{
    __shared__ unsigned long long sh[33];
    uint64_t base = (uint64_t)threadIdx.x * SCAN_ITEMS;
    unsigned long long v[SCAN_ITEMS];
    unsigned long long t = 0;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        v[i] = base + i < n ? data[base + i] : 0ull;
        t += v[i];
    }
    unsigned long long total;
    unsigned long long off = block_exclusive_scan(t, &total, sh);
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        if (base + i < n) data[base + i] = off;
        off += v[i];
    }
    if (threadIdx.x == 0 && total_out) *total_out = total;
}

__global__ void scan_apply(const unsigned long long* __restrict__ in, unsigned long long* __restrict__ out,
                           const unsigned long long* __restrict__ boff, uint64_t n)
{
    __shared__ unsigned long long sh[33];
    uint64_t base = (uint64_t)blockIdx.x * SCAN_TILE + (uint64_t)threadIdx.x * SCAN_ITEMS;
    unsigned long long v[SCAN_ITEMS];
    unsigned long long t = 0;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        v[i] = base + i < n ? in[base + i] : 0ull;
        t += v[i];
    }
    unsigned long long total;
    unsigned long long off = block_exclusive_scan(t, &total, sh) + boff[blockIdx.x];
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        if (base + i < n) out[base + i] = off;
        off += v[i];
    }
}

}  // namespace

size_t nups_scan_scratch_bytes(uint64_t n)
{
    size_t bytes = 0;
    uint64_t m = n;
    while (m > (uint64_t)SCAN_TILE) {
        m = (m + SCAN_TILE - 1) / SCAN_TILE;
        bytes += ((m * 8 + 255) / 256) * 256;
    }
    return bytes + 256;
}

nups_status nups_scan_u64(nups_store* s, const unsigned long long* d_in, unsigned long long* d_out, uint64_t n,
                          unsigned long long* d_total, char* scratch, cudaStream_t st)
{
    if (n == 0) {
        if (d_total) CK(cudaMemsetAsync(d_total, 0, 8, st));
        return NUPS_OK;
    }
    if (n <= (uint64_t)SCAN_TILE) {
        if (d_out != d_in) CK(cudaMemcpyAsync(d_out, d_in, n * 8, cudaMemcpyDeviceToDevice, st));
        scan_single_block<<<1, SCAN_THREADS, 0, st>>>(d_out, n, d_total);
        LAUNCH_CHECK(s);
        return NUPS_OK;
    }
    uint64_t nb = (n + SCAN_TILE - 1) / SCAN_TILE;
    unsigned long long* bsum = (unsigned long long*)scratch;
    char* rest = scratch + ((nb * 8 + 255) / 256) * 256;
    scan_block_sums<<<(unsigned)nb, SCAN_THREADS, 0, st>>>(d_in, bsum, n);
    LAUNCH_CHECK(s);
    nups_status rc = nups_scan_u64(s, bsum, bsum, nb, d_total, rest, st);
    if (rc != NUPS_OK) return rc;
    scan_apply<<<(unsigned)nb, SCAN_THREADS, 0, st>>>(d_in, d_out, bsum, n);
    LAUNCH_CHECK(s);
    return NUPS_OK;
}

// ---------------------------------------------------------------------------------------------
// Stable LSD radix sort, 8 bits per pass.  A block owns a tile of SORT_TILE consecutive pairs and
// walks it in rounds of one pair per thread, so that ranks inside the tile follow input order.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int SORT_THREADS = 256;
constexpr int SORT_ROUNDS = 8;
constexpr int SORT_TILE = SORT_THREADS * SORT_ROUNDS;
constexpr int RADIX = 256;

__global__ void sort_histogram(const unsigned long long* __restrict__ keys, uint64_t n, int shift,
                               unsigned long long* __restrict__ hist /* [RADIX][nblocks] */, unsigned nblocks)
{
    __shared__ unsigned h[RADIX];
    h[threadIdx.x] = 0;
    __syncthreads();
    uint64_t base = (uint64_t)blockIdx.x * SORT_TILE;
    for (int r = 0; r < SORT_ROUNDS; ++r) {
        uint64_t i = base + (uint64_t)r * SORT_THREADS + threadIdx.x;
        if (i < n) atomicAdd(&h[(keys[i] >> shift) & (RADIX - 1)], 1u);
    }
    __syncthreads();
    hist[(uint64_t)threadIdx.x * nblocks + blockIdx.x] = h[threadIdx.x];
}

__global__ void sort_scatter(const unsigned long long* __restrict__ keys, const uint32_t* __restrict__ vals,
                             unsigned long long* __restrict__ keys_out, uint32_t* __restrict__ vals_out, uint64_t n,
                             int shift, const unsigned long long* __restrict__ offs /* scanned hist */,
                             unsigned nblocks)
{
    __shared__ unsigned warp_cnt[SORT_THREADS / 32][RADIX];
    __shared__ unsigned long long running[RADIX];
    const unsigned lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    running[threadIdx.x] = offs[(uint64_t)threadIdx.x * nblocks + blockIdx.x];
    uint64_t base = (uint64_t)blockIdx.x * SORT_TILE;
    for (int r = 0; r < SORT_ROUNDS; ++r) {
        for (int w = 0; w < SORT_THREADS / 32; ++w) warp_cnt[w][threadIdx.x] = 0;
        __syncthreads();
        uint64_t i = base + (uint64_t)r * SORT_THREADS + threadIdx.x;
        bool ok = i < n;
        unsigned long long k = ok ? keys[i] : 0ull;
        unsigned d = ok ? (unsigned)((k >> shift) & (RADIX - 1)) : RADIX;   // RADIX = inactive
        unsigned m = __match_any_sync(0xFFFFFFFFu, d);
        unsigned rank = __popc(m & ((1u << lane) - 1u));
        if (ok && rank == 0) warp_cnt[warp][d] = __popc(m);
        __syncthreads();
        // thread d turns the per-warp counts of digit d into exclusive offsets
        {
            unsigned acc = 0;
            for (int w = 0; w < SORT_THREADS / 32; ++w) {
                unsigned c = warp_cnt[w][threadIdx.x];
                warp_cnt[w][threadIdx.x] = acc;
                acc += c;
            }
            __syncthreads();
            if (ok) {
                unsigned long long pos = running[d] + warp_cnt[warp][d] + rank;
                keys_out[pos] = k;
                vals_out[pos] = vals[i];
            }
            __syncthreads();
            running[threadIdx.x] += acc;
        }
        __syncthreads();
    }
}

}  // namespace

size_t nups_sort_scratch_bytes(uint64_t n)
{
    uint64_t nb = (n + SORT_TILE - 1) / SORT_TILE;
    if (nb == 0) nb = 1;
    size_t hist = ((size_t)RADIX * nb * 8 + 255) / 256 * 256;
    return hist + nups_scan_scratch_bytes((uint64_t)RADIX * nb) + 256;
}

nups_status nups_sort_pairs(nups_store* s, unsigned long long* k_in, uint32_t* v_in, unsigned long long* k_out,
                            uint32_t* v_out, uint64_t n, int bits, char* scratch, cudaStream_t st)
{
    if (n == 0) return NUPS_OK;
    unsigned nb = (unsigned)((n + SORT_TILE - 1) / SORT_TILE);
    unsigned long long* hist = (unsigned long long*)scratch;
    char* scan_scratch = scratch + ((size_t)RADIX * nb * 8 + 255) / 256 * 256;
    int passes = (bits + 7) / 8;
    if (passes < 1) passes = 1;
    if (!(passes & 1)) {
        // every pass flips the buffers; an even number of passes would end in the caller's input
        // buffers, so start from a copy in the output buffers instead
        CK(cudaMemcpyAsync(k_out, k_in, n * 8, cudaMemcpyDeviceToDevice, st));
        CK(cudaMemcpyAsync(v_out, v_in, n * 4, cudaMemcpyDeviceToDevice, st));
        unsigned long long* tk = k_in; k_in = k_out; k_out = tk;
        uint32_t* tv = v_in; v_in = v_out; v_out = tv;
    }
    for (int p = 0; p < passes; ++p) {
        int shift = 8 * p;
        sort_histogram<<<nb, SORT_THREADS, 0, st>>>(k_in, n, shift, hist, nb);
        LAUNCH_CHECK(s);
        nups_status rc = nups_scan_u64(s, hist, hist, (uint64_t)RADIX * nb, nullptr, scan_scratch, st);
        if (rc != NUPS_OK) return rc;
        sort_scatter<<<nb, SORT_THREADS, 0, st>>>(k_in, v_in, k_out, v_out, n, shift, hist, nb);
        LAUNCH_CHECK(s);
        unsigned long long* tk = k_in; k_in = k_out; k_out = tk;
        uint32_t* tv = v_in; v_in = v_out; v_out = tv;
    }
    return NUPS_OK;
}
