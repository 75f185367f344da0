// Sampling access: register_distribution (alias table built on the device), PrepareSample and
// PullSample under the four conformity levels.  NuPS Sections 4.3, 4.4.
#include <string.h>

#include "nups_internal.cuh"

static inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// ---------------------------------------------------------------------------------------------
// Alias table.  n buckets of capacity W = sum w; item j has mass n*w[j]; "lights" have mass < W.
// Lights are topped up by the heavies in index order, and a heavy whose remainder drops below W
// is itself topped up by the next heavy.  With D(a) the running sum of the lights' deficits and
// S(h) the running sum of the heavies' surpluses (both in index order):
//   light a is filled by the first heavy h with S(h) >= D(a-1);
//   heavy h turns light right after the first light a with D(a) > S(h); it keeps
//   W + S(h) - D(a) and is filled by heavy h+1; a heavy that never turns light keeps W.
// ---------------------------------------------------------------------------------------------
__global__ void weight_sum_kernel(const uint32_t* __restrict__ w, uint64_t n, DevStat* st)
{
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    unsigned long long sum = 0;
    for (; i < n; i += stride) sum += w[i];
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
    if ((threadIdx.x & 31) == 0 && sum) atomicAdd(&st->tmp[0], sum);
}

__global__ void alias_classify_kernel(const uint32_t* __restrict__ w, uint64_t n, unsigned long long W,
                                      unsigned long long* __restrict__ lflag, unsigned long long* __restrict__ dfl,
                                      unsigned long long* __restrict__ sfl)
{
    uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    unsigned long long mass = n * (unsigned long long)w[j];
    bool light = mass < W;
    lflag[j] = light ? 1ull : 0ull;
    dfl[j] = light ? W - mass : 0ull;
    sfl[j] = light ? 0ull : mass - W;
}

__global__ void alias_rank_kernel(const uint32_t* __restrict__ w, uint64_t n, unsigned long long W,
                                  const unsigned long long* __restrict__ lrank, const unsigned long long* __restrict__ dex,
                                  const unsigned long long* __restrict__ sex, unsigned long long nL,
                                  unsigned long long* __restrict__ inc /* D at [0,nL), S at [nL,n) */,
                                  uint32_t* __restrict__ hidx)
{
    uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    unsigned long long mass = n * (unsigned long long)w[j];
    unsigned long long a = lrank[j];
    if (mass < W) inc[a] = dex[j] + (W - mass);
    else {
        unsigned long long h = j - a;
        inc[nL + h] = sex[j] + (mass - W);
        hidx[h] = (uint32_t)j;
    }
}

__global__ void alias_fill_kernel(const uint32_t* __restrict__ w, uint64_t n, unsigned long long W,
                                  const unsigned long long* __restrict__ lrank, const unsigned long long* __restrict__ dex,
                                  unsigned long long nL, const unsigned long long* __restrict__ inc,
                                  const uint32_t* __restrict__ hidx, AliasEntry* __restrict__ table)
{
    uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    const unsigned long long* D = inc;
    const unsigned long long* S = inc + nL;
    const unsigned long long nH = n - nL;
    unsigned long long mass = n * (unsigned long long)w[j];
    AliasEntry e;
    e.pad = 0;
    if (mass < W) {
        unsigned long long target = dex[j];          // D(a-1)
        unsigned long long lo = 0, hi = nH;          // first h with S[h] >= target
        while (lo < hi) {
            unsigned long long mid = (lo + hi) >> 1;
            if (S[mid] >= target) hi = mid; else lo = mid + 1;
        }
        e.thr = mass;
        e.alias = hidx[lo < nH ? lo : nH - 1];
    } else {
        unsigned long long h = j - lrank[j];
        unsigned long long Sh = S[h];
        unsigned long long lo = 0, hi = nL;          // first a with D[a] > Sh
        while (lo < hi) {
            unsigned long long mid = (lo + hi) >> 1;
            if (D[mid] > Sh) hi = mid; else lo = mid + 1;
        }
        if (lo < nL && h + 1 < nH) {
            e.thr = W + Sh - D[lo];
            e.alias = hidx[h + 1];
        } else {
            e.thr = W;
            e.alias = (uint32_t)j;
        }
    }
    table[j] = e;
}

__global__ void alias_unpack_kernel(const AliasEntry* __restrict__ table, uint64_t n, unsigned long long* thr,
                                    uint32_t* alias)
{
    uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    thr[j] = table[j].thr;
    alias[j] = table[j].alias;
}

extern "C" nups_status nups_register_distribution(nups_store* s, uint32_t key_base, const uint32_t* d_weights,
                                                  uint64_t n, int level, uint32_t U, uint32_t G, uint64_t seed,
                                                  int32_t* h_dist_out, void* stream)
{
    if (!s || !h_dist_out) return NUPS_EINVAL;
    if (n == 0 || (uint64_t)key_base + n > s->num_keys) return NUPS_EINVAL;
    if (level < NUPS_CONFORM || level > NUPS_NONCONFORM) return NUPS_EINVAL;
    bool reuse = level == NUPS_BOUNDED || level == NUPS_LONGTERM;
    if (reuse && (U == 0 || G == 0 || G > NUPS_MAX_POOL)) return NUPS_EINVAL;
    if ((level == NUPS_LONGTERM || level == NUPS_NONCONFORM) && !s->owner) return NUPS_ESTATE;
    int id = -1;
    for (int i = 0; i < NUPS_MAX_DISTS; ++i) if (!s->dist[i].used) { id = i; break; }
    if (id < 0) return NUPS_ENOMEM;
    cudaStream_t st = (cudaStream_t)stream;
    Dist d;
    memset(&d, 0, sizeof(d));
    d.key_base = key_base; d.n = n; d.level = level; d.U = U; d.G = G; d.seed = seed;
    if (!d_weights) d.uniform = 1;
    else {
        CK(cudaMemsetAsync(&s->st->tmp[0], 0, 8, st));
        weight_sum_kernel<<<grid_for(n, 256, (unsigned)s->sm_count * 8), 256, 0, st>>>(d_weights, n, s->st);
        LAUNCH_CHECK(s);
        unsigned long long W = 0;
        CK(cudaMemcpyAsync(&W, &s->st->tmp[0], 8, cudaMemcpyDeviceToHost, st));
        CK(cudaStreamSynchronize(st));
        if (W == 0) return NUPS_EINVAL;
        unsigned __int128 nW = (unsigned __int128)W * n;
        if (nW >> 64) return NUPS_EINVAL;
        d.W = W;
        size_t need = 4 * align256(n * 8) + align256(n * 4) + nups_scan_scratch_bytes(n) + 256;
        char* sc;
        nups_status rc = nups_scratch(s, need, &sc);
        if (rc != NUPS_OK) return rc;
        unsigned long long* lrank = (unsigned long long*)sc; sc += align256(n * 8);
        unsigned long long* dex = (unsigned long long*)sc; sc += align256(n * 8);
        unsigned long long* sex = (unsigned long long*)sc; sc += align256(n * 8);
        unsigned long long* inc = (unsigned long long*)sc; sc += align256(n * 8);
        uint32_t* hidx = (uint32_t*)sc; sc += align256(n * 4);
        unsigned long long* d_nL = (unsigned long long*)sc; sc += 256;
        if (cudaMalloc(&d.table, n * sizeof(AliasEntry)) != cudaSuccess) { cudaGetLastError(); return NUPS_ENOMEM; }
        unsigned g = grid_for(n, 256);
        alias_classify_kernel<<<g, 256, 0, st>>>(d_weights, n, W, lrank, dex, sex);
        LAUNCH_CHECK(s);
        rc = nups_scan_u64(s, lrank, lrank, n, d_nL, sc, st);
        if (rc == NUPS_OK) rc = nups_scan_u64(s, dex, dex, n, nullptr, sc, st);
        if (rc == NUPS_OK) rc = nups_scan_u64(s, sex, sex, n, nullptr, sc, st);
        if (rc != NUPS_OK) { cudaFree(d.table); return rc; }
        unsigned long long nL = 0;
        CK(cudaMemcpyAsync(&nL, d_nL, 8, cudaMemcpyDeviceToHost, st));
        CK(cudaStreamSynchronize(st));
        alias_rank_kernel<<<g, 256, 0, st>>>(d_weights, n, W, lrank, dex, sex, nL, inc, hidx);
        LAUNCH_CHECK(s);
        alias_fill_kernel<<<g, 256, 0, st>>>(d_weights, n, W, lrank, dex, nL, inc, hidx, (AliasEntry*)d.table);
        LAUNCH_CHECK(s);
        CK(cudaStreamSynchronize(st));
    }
    if (cudaMalloc(&d.off, 2 * s->R * 8) != cudaSuccess) { cudaGetLastError(); cudaFree(d.table); return NUPS_ENOMEM; }
    CK(cudaMemsetAsync(d.off, 0, 2 * s->R * 8, st));
    CK(cudaStreamSynchronize(st));
    d.used = 1;
    s->dist[id] = d;
    *h_dist_out = id;
    return NUPS_OK;
}

extern "C" nups_status nups_get_alias_table(nups_store* s, int32_t dist, uint64_t* d_thr_out, uint32_t* d_alias_out,
                                            uint64_t* h_W_out, void* stream)
{
    if (!s || dist < 0 || dist >= NUPS_MAX_DISTS || !s->dist[dist].used) return NUPS_EINVAL;
    Dist& d = s->dist[dist];
    if (h_W_out) *h_W_out = d.W;
    if (d.uniform) return d_thr_out || d_alias_out ? NUPS_EINVAL : NUPS_OK;
    if (d_thr_out && d_alias_out) {
        alias_unpack_kernel<<<grid_for(d.n, 256), 256, 0, (cudaStream_t)stream>>>((const AliasEntry*)d.table, d.n,
                                                                              (unsigned long long*)d_thr_out, d_alias_out);
        LAUNCH_CHECK(s);
    }
    return NUPS_OK;
}

// ---------------------------------------------------------------------------------------------
// Draws
// ---------------------------------------------------------------------------------------------
struct DrawParams {
    const AliasEntry* table;
    unsigned long long n, W, seed;
    uint32_t key_base, U, G;
    int uniform;
};

static DrawParams draw_params(const Dist& d)
{
    DrawParams p;
    p.table = (const AliasEntry*)d.table; p.n = d.n; p.W = d.W; p.seed = d.seed;
    p.key_base = d.key_base; p.U = d.U; p.G = d.G; p.uniform = d.uniform;
    return p;
}

// one iid draw from pi: position `pos` of worker q's stream; 64 bits pick the bucket, 64 bits the
// point inside it
__device__ __forceinline__ uint32_t draw_iid(const DrawParams& p, uint32_t q, unsigned long long pos)
{
    uint32_t x[4];
    philox_at(p.seed, pos, q, 0, 0, x);
    unsigned long long a = (unsigned long long)x[0] | ((unsigned long long)x[1] << 32);
    unsigned long long b = (unsigned long long)x[2] | ((unsigned long long)x[3] << 32);
    unsigned long long j = __umul64hi(a, p.n);
    if (!p.uniform) {
        AliasEntry e = p.table[j];
        if (!(__umul64hi(b, p.W) < e.thr)) j = e.alias;
    }
    return p.key_base + (uint32_t)j;
}

// Handle buffer layout (device): start[R] (u64) | keys[N] (u32) | post[N] (u32) | state[R] (uint4)
struct HandleView {
    unsigned long long* start;
    uint32_t* keys;
    uint32_t* post;
    uint4* state;      // LONG-TERM per sub-handle: x = walk position, y = postponed head, z = postponed tail
};
static size_t handle_bytes(uint64_t N, uint32_t R, int level)
{
    size_t b = align256((size_t)R * 8) + align256(N * 4);
    if (level == NUPS_LONGTERM) b += align256(N * 4) + align256((size_t)R * 16);
    return b;
}
static HandleView handle_view(char* buf, uint64_t N, uint32_t R)
{
    HandleView h;
    h.start = (unsigned long long*)buf; buf += align256((size_t)R * 8);
    h.keys = (uint32_t*)buf; buf += align256(N * 4);
    h.post = (uint32_t*)buf; buf += align256(N * 4);
    h.state = (uint4*)buf;
    return h;
}

__global__ void handle_begin_kernel(const unsigned long long* off_cur, unsigned long long* off_next, HandleView h,
                                    uint64_t N, uint32_t R, int longterm)
{
    uint32_t q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= R) return;
    unsigned long long size = chunk_begin(q + 1, N, R) - chunk_begin(q, N, R);
    h.start[q] = off_cur[q];
    off_next[q] = off_cur[q] + size;
    if (longterm) h.state[q] = make_uint4(0u, 0u, 0u, 0u);
}

__global__ void draw_iid_kernel(DrawParams p, HandleView h, uint64_t N, uint32_t R)
{
    uint64_t o = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (o >= N) return;
    uint32_t q = chunk_of_pos(o, N, R);
    h.keys[o] = draw_iid(p, q, h.start[q] + (o - chunk_begin(q, N, R)));
}

// Pooled reuse: pool `pl` of a worker holds G iid draws and is walked U times, each pass in a fresh
// Fisher-Yates order.  Stream position s lies in pass number s / G overall (pool = pass / U).
// One block produces one pass of one worker.
__global__ void draw_reuse_kernel(DrawParams p, HandleView h, uint64_t N, uint32_t R)
{
    __shared__ uint32_t pool[NUPS_MAX_POOL];
    __shared__ uint32_t perm[NUPS_MAX_POOL];
    __shared__ uint32_t xs[NUPS_MAX_POOL];
    const uint32_t q = blockIdx.y, G = p.G;
    const unsigned long long b0 = chunk_begin(q, N, R), size = chunk_begin(q + 1, N, R) - b0;
    if (size == 0) return;
    const unsigned long long s0 = h.start[q], s1 = s0 + size;
    const unsigned long long pass = s0 / G + blockIdx.x;
    if (pass * G >= s1) return;
    const unsigned long long pl = pass / p.U;
    for (uint32_t m = threadIdx.x; m < G; m += blockDim.x) {
        pool[m] = draw_iid(p, q, pl * G + m);
        perm[m] = m;
    }
    // random words of the shuffle: word d of the pass's Philox stream (purpose 1), four per block
    for (uint32_t blk = threadIdx.x; blk * 4 < G - 1; blk += blockDim.x) {
        uint32_t x[4];
        philox_at(p.seed, pass, q, 1, blk, x);
        for (int k = 0; k < 4; ++k)
            if (blk * 4 + k < G - 1) xs[blk * 4 + k] = x[k];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (uint32_t i = G - 1; i >= 1; --i) {
            uint32_t r = __umulhi(xs[G - 1 - i], i + 1);
            uint32_t t = perm[i]; perm[i] = perm[r]; perm[r] = t;
        }
    }
    __syncthreads();
    for (uint32_t j = threadIdx.x; j < G; j += blockDim.x) {
        unsigned long long sp = pass * G + j;
        if (sp >= s0 && sp < s1) h.keys[b0 + (sp - s0)] = pool[perm[j]];
    }
}

// PrepareSample localizes the sampled keys to the sub-handle's worker
__global__ void localize_handle_kernel(View v, const uint32_t* __restrict__ keys, uint64_t N, uint32_t* req,
                                       uint64_t req_cap)
{
    uint64_t o = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool in = o < N;
    queue_localize(v, in, in ? keys[o] : 0u, in ? chunk_of_pos(o, N, v.R) : 0u, req, req_cap);
}

static nups_status prepare_internal(nups_store* s, int32_t dist, uint64_t N, int* slot_out, cudaStream_t st)
{
    if (dist < 0 || dist >= NUPS_MAX_DISTS || !s->dist[dist].used || N == 0 || N >= (1ull << 32)) return NUPS_EINVAL;
    if (s->ahead_dist == dist) {
        nups_status rw = nups_sample_ahead_rewind(s, st);       // samples drawn ahead for the steps go back
        if (rw != NUPS_OK) return rw;
    }
    Dist& d = s->dist[dist];
    size_t need = handle_bytes(N, s->R, d.level);
    int id = -1;
    for (int i = 0; i < NUPS_MAX_HANDLES && id < 0; ++i)
        if (!s->handle[i].used && s->handle[i].cap >= need) id = i;      // reuse a released buffer
    for (int i = 0; i < NUPS_MAX_HANDLES && id < 0; ++i)
        if (!s->handle[i].used && s->handle[i].cap == 0) id = i;
    for (int i = 0; i < NUPS_MAX_HANDLES && id < 0; ++i)
        if (!s->handle[i].used) id = i;
    if (id < 0) return NUPS_ENOMEM;
    Handle& h = s->handle[id];
    if (h.cap < need) {
        if (h.buf) CK(cudaFree(h.buf));
        h.buf = nullptr; h.cap = 0;
        size_t want = need + need / 4;
        if (cudaMalloc(&h.buf, want) != cudaSuccess) { cudaGetLastError(); return NUPS_ENOMEM; }
        h.cap = want;
    }
    bool reuse = d.level == NUPS_BOUNDED || d.level == NUPS_LONGTERM;
    bool loc = s->owner && d.level != NUPS_NONCONFORM;
    if (loc || d.level == NUPS_LONGTERM) {
        nups_status rc = nups_req_reserve(s, N);
        if (rc != NUPS_OK) return rc;
    }
    HandleView hv = handle_view(h.buf, N, s->R);
    DrawParams p = draw_params(d);
    handle_begin_kernel<<<grid_for(s->R, 64), 64, 0, st>>>(d.off + (size_t)d.cur * s->R, d.off + (size_t)(d.cur ^ 1) * s->R,
                                                           hv, N, s->R, d.level == NUPS_LONGTERM);
    LAUNCH_CHECK(s);
    d.cur ^= 1;
    if (reuse) {
        uint64_t max_size = (N + s->R - 1) / s->R;
        unsigned passes = (unsigned)(max_size / d.G + 2);
        unsigned threads = ((d.G + 31) / 32) * 32;
        if (threads > 256) threads = 256;
        draw_reuse_kernel<<<dim3(passes, s->R), threads, 0, st>>>(p, hv, N, s->R);
    } else {
        draw_iid_kernel<<<grid_for(N, 256), 256, 0, st>>>(p, hv, N, s->R);
    }
    LAUNCH_CHECK(s);
    if (loc) {
        localize_handle_kernel<<<grid_for(N, 256), 256, 0, st>>>(nups_view(s), hv.keys, N, s->req_keys, s->req_cap);
        LAUNCH_CHECK(s);
        nups_status rc = nups_localize_apply(s, N, st);
        if (rc != NUPS_OK) return rc;
    }
    h.used = 1; h.dist = dist; h.N = N; h.cursor = 0;
    *slot_out = id;
    return NUPS_OK;
}

extern "C" nups_status nups_prepare_sample(nups_store* s, int32_t dist, uint64_t N, nups_handle* h_out, void* stream)
{
    if (!s || !h_out) return NUPS_EINVAL;
    int id = -1;
    nups_status rc = prepare_internal(s, dist, N, &id, (cudaStream_t)stream);
    if (rc == NUPS_OK) *h_out = id;
    return rc;
}

// ---------------------------------------------------------------------------------------------
// PullSample
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void count_sample(const View& v, uint32_t key, bool emitted)
{
    if (!v.count) return;
    const unsigned lane = threadIdx.x & 31;
    bool hot = emitted && key_is_hot(v, key);
    if (emitted) atomicAdd(v.cnt + key, 1ull);
    unsigned hot_m = __ballot_sync(0xFFFFFFFFu, emitted && hot);
    unsigned cold_m = __ballot_sync(0xFFFFFFFFu, emitted && !hot);
    if (lane == 0) {
        if (hot_m) atomicAdd(&v.st->hot_hits, (unsigned long long)__popc(hot_m));
        if (cold_m) atomicAdd(&v.st->cold_hits, (unsigned long long)__popc(cold_m));
    }
}

// independent draws / pooled reuse: the keys were fixed at PrepareSample.
// local sampling: first key local to the worker at or after the candidate.
__global__ void emit_kernel(View v, DrawParams p, HandleView h, uint64_t N, uint64_t cursor, uint64_t n, int local_only,
                            uint32_t* __restrict__ out)
{
    uint64_t o = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    bool in = o < n;
    uint32_t k = 0;
    if (in) {
        uint64_t pos = cursor + o;
        k = h.keys[pos];
        if (local_only) {
            uint32_t q = chunk_of_pos(pos, N, v.R);
            uint32_t k0 = k;
            for (uint32_t probe = 0; probe < NUPS_LOCAL_PROBES; ++probe) {
                uint32_t cand = p.key_base + (uint32_t)(((unsigned long long)(k0 - p.key_base) + probe) % p.n);
                if (key_is_local(v, q, cand)) { k = cand; break; }
            }
        }
        out[o] = k;
    }
    count_sample(v, k, in);
}

// reuse with postponing: one block walks one sub-handle.  Entries not yet postponed are taken in
// order; a local one is emitted, a non-local one is queued for re-localization and appended to the
// sub-handle's postponed queue; when the fresh entries run out the postponed ones are emitted.
constexpr int LT_THREADS = 1024;
constexpr int LT_ITEMS = 4;                 // consecutive list entries per thread and round

__global__ void __launch_bounds__(LT_THREADS)
longterm_kernel(View v, HandleView h, uint64_t N, uint64_t cursor, uint64_t n, uint32_t q_first,
                uint32_t* __restrict__ out, uint32_t* req, uint64_t req_cap)
{
    __shared__ unsigned warp_tot[LT_THREADS / 32];
    __shared__ unsigned sh_consumed, sh_local;
    const uint32_t q = q_first + blockIdx.x;
    const unsigned tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint64_t b0 = chunk_begin(q, N, v.R), b1 = chunk_begin(q + 1, N, v.R);
    const uint64_t lo = max(b0, cursor), hi = min(b1, cursor + n);
    if (lo >= hi) return;
    const uint64_t take = hi - lo, size = b1 - b0;
    const uint64_t out_base = lo - cursor;
    uint4 stt = h.state[q];
    uint64_t oc = stt.x, ph = stt.y, pt = stt.z, emitted = 0;
    while (emitted < take && oc < size) {
        // a round looks at LT_THREADS * LT_ITEMS fresh entries in list order: thread t owns entries
        // t * LT_ITEMS .. t * LT_ITEMS + LT_ITEMS - 1 of the round
        uint32_t key[LT_ITEMS];
        bool have[LT_ITEMS], loc[LT_ITEMS];
        unsigned mine = 0;
#pragma unroll
        for (int k = 0; k < LT_ITEMS; ++k) {
            const uint64_t i = oc + (uint64_t)tid * LT_ITEMS + k;
            have[k] = i < size;
            key[k] = have[k] ? h.keys[b0 + i] : 0u;
            loc[k] = have[k] && key_is_local(v, q, key[k]);
            mine += loc[k] ? 1u : 0u;
        }
        // exclusive count of local entries before this thread's first entry
        unsigned inc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
            if (lane >= (unsigned)o) inc += y;
        }
        if (lane == 31) warp_tot[warp] = inc;
        if (tid == 0) { sh_consumed = 0; sh_local = 0; }
        __syncthreads();
        unsigned excl = inc - mine;
        for (unsigned w = 0; w < warp; ++w) excl += warp_tot[w];
        const uint64_t need = take - emitted;
        unsigned nc = 0, nl = 0;
#pragma unroll
        for (int k = 0; k < LT_ITEMS; ++k) {
            // the walk stops right after the need-th local entry: an entry is reached iff fewer than
            // `need` local entries lie before it
            const bool consumed = have[k] && excl < need;
            if (consumed) {
                if (loc[k]) out[out_base + emitted + excl] = key[k];
                else {
                    h.post[b0 + pt + ((uint64_t)tid * LT_ITEMS + k - excl)] = key[k];     // non-local entries before it
                    atomicMax(v.pending + key[k], (int)q);
                    const unsigned long long at = atomicAdd(&v.st->req_count, 1ull);
                    if (at < req_cap) req[at] = key[k];
                }
                nc++;
                nl += loc[k] ? 1u : 0u;
            }
            count_sample(v, key[k], consumed && loc[k]);
            excl += loc[k] ? 1u : 0u;
        }
        for (int o = 16; o > 0; o >>= 1) {
            nc += __shfl_xor_sync(0xFFFFFFFFu, nc, o);
            nl += __shfl_xor_sync(0xFFFFFFFFu, nl, o);
        }
        if (lane == 0) { atomicAdd(&sh_consumed, nc); atomicAdd(&sh_local, nl); }
        __syncthreads();
        const unsigned tc = sh_consumed, tl = sh_local;
        emitted += tl; pt += tc - tl; oc += tc;
        __syncthreads();
    }
    __syncthreads();
    if (emitted < take) {
        const uint64_t cnt = take - emitted;
        for (uint64_t i = tid; i < ((cnt + LT_THREADS - 1) / LT_THREADS) * LT_THREADS; i += LT_THREADS) {
            const bool in = i < cnt;
            const uint32_t key = in ? h.post[b0 + ph + i] : 0u;
            if (in) out[out_base + emitted + i] = key;
            count_sample(v, key, in);
        }
        ph += cnt;
    }
    if (tid == 0) h.state[q] = make_uint4((unsigned)oc, (unsigned)ph, (unsigned)pt, 0u);
}

static nups_status pull_internal(nups_store* s, int id, uint64_t n, uint32_t* d_keys_out, float* d_vals_out,
                                 cudaStream_t st)
{
    Handle& h = s->handle[id];
    Dist& d = s->dist[h.dist];
    if (n > h.N - h.cursor) return NUPS_ESTATE;
    if (n == 0) return NUPS_OK;
    View v = nups_view(s);
    HandleView hv = handle_view(h.buf, h.N, s->R);
    DrawParams p = draw_params(d);
    if (d.level == NUPS_LONGTERM) {
        // sub-handles overlapped by [cursor, cursor + n)
        uint32_t qf = 0, ql = 0;
        for (uint32_t q = 0; q < s->R; ++q) {
            uint64_t b0 = ((uint64_t)q * h.N) / s->R, b1 = ((uint64_t)(q + 1) * h.N) / s->R;
            if (b0 <= h.cursor && h.cursor < b1) qf = q;
            if (b0 <= h.cursor + n - 1 && h.cursor + n - 1 < b1) ql = q;
        }
        longterm_kernel<<<ql - qf + 1, LT_THREADS, 0, st>>>(v, hv, h.N, h.cursor, n, qf, d_keys_out, s->req_keys, s->req_cap);
        LAUNCH_CHECK(s);
        nups_status rc = nups_localize_apply(s, h.N, st);
        if (rc != NUPS_OK) return rc;
    } else {
        emit_kernel<<<grid_for(n, 256), 256, 0, st>>>(v, p, hv, h.N, h.cursor, n, d.level == NUPS_NONCONFORM, d_keys_out);
        LAUNCH_CHECK(s);
    }
    if (d_vals_out) {
        nups_status rc = nups_gather_internal(s, d_keys_out, n, d_vals_out, nullptr, 1, h.cursor, h.N, 0, st);
        if (rc != NUPS_OK) return rc;
    }
    h.cursor += n;
    if (h.cursor == h.N) h.used = 0;       // released; the buffer stays for the next handle
    return NUPS_OK;
}

extern "C" nups_status nups_pull_sample(nups_store* s, nups_handle handle, uint64_t n, uint32_t* d_keys_out,
                                        float* d_vals_out, void* stream)
{
    if (!s || handle < 0 || handle >= NUPS_MAX_HANDLES || !s->handle[handle].used) return NUPS_EINVAL;
    if (n && !d_keys_out) return NUPS_EINVAL;
    return pull_internal(s, (int)handle, n, d_keys_out, d_vals_out, (cudaStream_t)stream);
}

// ---------------------------------------------------------------------------------------------
// PrepareSample + one full PullSample (keys only) in a single launch, for the workload steps: the
// same keys as the handle path gives, written straight to `out`.  Stream offsets are read from one
// half of the distribution's offset array and the advanced offsets written to the other half.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void direct_tail(const View& v, uint32_t key, uint32_t q, bool in, bool localize, uint32_t* req,
                                            uint64_t req_cap)
{
    count_sample(v, key, in);
    if (localize) queue_localize(v, in, key, q, req, req_cap);
}

// blockIdx.y (iid) / blockIdx.z (reuse) = batch: `batches` handles of N samples each are drawn back to back,
// exactly as that many separate calls would draw them; batch b goes to out + b * N.
__global__ void draw_direct_iid_kernel(View v, DrawParams p, const unsigned long long* off_cur,
                                       unsigned long long* off_next, uint64_t N, uint32_t batches, int local_only,
                                       int localize, uint32_t* __restrict__ out, uint32_t* req, uint64_t req_cap)
{
    const uint64_t o = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t bt = blockIdx.y;
    const bool in = o < N;
    uint32_t k = 0, q = 0;
    out += (uint64_t)bt * N;
    if (in) {
        q = chunk_of_pos(o, N, v.R);
        const unsigned long long size = chunk_begin(q + 1, N, v.R) - chunk_begin(q, N, v.R);
        k = draw_iid(p, q, off_cur[q] + (unsigned long long)bt * size + (o - chunk_begin(q, N, v.R)));
        if (local_only) {
            const uint32_t k0 = k;
            for (uint32_t probe = 0; probe < NUPS_LOCAL_PROBES; ++probe) {
                uint32_t cand = p.key_base + (uint32_t)(((unsigned long long)(k0 - p.key_base) + probe) % p.n);
                if (key_is_local(v, q, cand)) { k = cand; break; }
            }
        }
        out[o] = k;
    }
    direct_tail(v, k, q, in, localize != 0, req, req_cap);
    if (blockIdx.x == 0 && blockIdx.y == 0)
        for (uint32_t w = threadIdx.x; w < v.R; w += blockDim.x)
            off_next[w] = off_cur[w] + (unsigned long long)batches * (chunk_begin(w + 1, N, v.R) - chunk_begin(w, N, v.R));
}

__global__ void draw_direct_reuse_kernel(View v, DrawParams p, const unsigned long long* off_cur,
                                         unsigned long long* off_next, uint64_t N, uint32_t batches, int localize,
                                         uint32_t* __restrict__ out, uint32_t* req, uint64_t req_cap)
{
    __shared__ uint32_t pool[NUPS_MAX_POOL];
    __shared__ uint32_t perm[NUPS_MAX_POOL];
    __shared__ uint32_t xs[NUPS_MAX_POOL];
    const uint32_t q = blockIdx.y, G = p.G, R = v.R;
    if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0)
        for (uint32_t w = threadIdx.x; w < R; w += blockDim.x)
            off_next[w] = off_cur[w] + (unsigned long long)batches * (chunk_begin(w + 1, N, R) - chunk_begin(w, N, R));
    const unsigned long long b0 = chunk_begin(q, N, R), size = chunk_begin(q + 1, N, R) - b0;
    if (size == 0) return;
    out += (uint64_t)blockIdx.z * N;
    const unsigned long long s0 = off_cur[q] + (unsigned long long)blockIdx.z * size, s1 = s0 + size;
    const unsigned long long pass = s0 / G + blockIdx.x;
    if (pass * G >= s1) return;
    const unsigned long long pl = pass / p.U;
    for (uint32_t m = threadIdx.x; m < G; m += blockDim.x) {
        pool[m] = draw_iid(p, q, pl * G + m);
        perm[m] = m;
    }
    for (uint32_t blk = threadIdx.x; blk * 4 < G - 1; blk += blockDim.x) {
        uint32_t x[4];
        philox_at(p.seed, pass, q, 1, blk, x);
        for (int k = 0; k < 4; ++k)
            if (blk * 4 + k < G - 1) xs[blk * 4 + k] = x[k];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (uint32_t i = G - 1; i >= 1; --i) {
            uint32_t r = __umulhi(xs[G - 1 - i], i + 1);
            uint32_t t = perm[i]; perm[i] = perm[r]; perm[r] = t;
        }
    }
    __syncthreads();
    const uint32_t rounds = (G + blockDim.x - 1) / blockDim.x;
    for (uint32_t rd = 0; rd < rounds; ++rd) {           // whole warps take every round: the tail ballots
        const uint32_t j = rd * blockDim.x + threadIdx.x;
        const unsigned long long sp = pass * G + j;
        const bool in = j < G && sp >= s0 && sp < s1;
        uint32_t k = 0;
        if (in) {
            k = pool[perm[j]];
            out[b0 + (sp - s0)] = k;
        }
        direct_tail(v, k, q, in, localize != 0, req, req_cap);
    }
}

// Sample-ahead for the workload steps.  The sample streams are a pure function of (seed, worker,
// position), so the negatives of the next NUPS_SAMPLE_AHEAD steps can be drawn in one launch and
// handed out one batch per step.  If anything else touches the distribution before they are used up
// (PrepareSample, a step with another size), the stream offsets are rewound by what was not handed out,
// so every sample sequence is the same as without sample-ahead.  Only used where drawing early has no
// other effect: fast mode, no access counting, no ownership tracking.
__global__ void rewind_kernel(unsigned long long* off, uint64_t N, uint32_t R, uint32_t batches)
{
    const uint32_t q = threadIdx.x;
    if (q < R) off[q] -= (unsigned long long)batches * (chunk_begin(q + 1, N, R) - chunk_begin(q, N, R));
}

nups_status nups_sample_ahead_rewind(nups_store* s, cudaStream_t st)
{
    if (s->ahead_dist < 0) return NUPS_OK;
    const uint32_t left = s->ahead_total - s->ahead_next;
    if (left) {
        Dist& d = s->dist[s->ahead_dist];
        rewind_kernel<<<1, 256, 0, st>>>(d.off + (size_t)d.cur * s->R, s->ahead_N, s->R, left);
        LAUNCH_CHECK(s);
    }
    s->ahead_dist = -1;
    return NUPS_OK;
}

// negatives of a workload step: one handle of N samples, pulled at once into library memory
nups_status nups_draw_negatives(nups_store* s, int32_t dist, uint64_t N, cudaStream_t st)
{
    s->last_negs_n = 0;
    if (N == 0) return NUPS_OK;
    if (dist < 0 || dist >= NUPS_MAX_DISTS || !s->dist[dist].used || N >= (1ull << 32)) return NUPS_EINVAL;
    // a batch drawn ahead for exactly this request?
    if (s->ahead_dist == dist && s->ahead_N == N && s->ahead_next < s->ahead_total) {
        s->last_negs = s->negs_buf + (uint64_t)s->ahead_next * N;
        s->last_negs_n = N;
        s->ahead_next++;
        return NUPS_OK;
    }
    nups_status rc = nups_sample_ahead_rewind(s, st);
    if (rc != NUPS_OK) return rc;
    Dist& d = s->dist[dist];
    const bool plain = d.level == NUPS_CONFORM || d.level == NUPS_BOUNDED;
    const uint32_t batches = (plain && !s->cfg.deterministic && !s->cfg.count_accesses && !s->owner &&
                              N * NUPS_SAMPLE_AHEAD < (1ull << 28)) ? NUPS_SAMPLE_AHEAD : 1;
    if (N * batches > s->negs_cap) {
        if (s->negs_buf) CK(cudaFree(s->negs_buf));
        s->negs_buf = nullptr; s->negs_cap = 0;
        uint64_t want = N * batches + N / 4;
        if (cudaMalloc(&s->negs_buf, want * 4) != cudaSuccess) { cudaGetLastError(); return NUPS_ENOMEM; }
        s->negs_cap = want;
    }
    s->last_negs = s->negs_buf;
    if (d.level == NUPS_LONGTERM) {
        // postponing needs the handle's walk state: PrepareSample, then one full PullSample
        int id = -1;
        rc = prepare_internal(s, dist, N, &id, st);
        if (rc != NUPS_OK) return rc;
        rc = pull_internal(s, id, N, s->last_negs, nullptr, st);
        if (rc != NUPS_OK) return rc;
        s->last_negs_n = N;
        return NUPS_OK;
    }
    const int localize = s->owner && d.level != NUPS_NONCONFORM;
    if (localize) {
        rc = nups_req_reserve(s, N);
        if (rc != NUPS_OK) return rc;
    }
    View v = nups_view(s);
    DrawParams p = draw_params(d);
    const unsigned long long* off_cur = d.off + (size_t)d.cur * s->R;
    unsigned long long* off_next = d.off + (size_t)(d.cur ^ 1) * s->R;
    if (d.level == NUPS_BOUNDED) {
        uint64_t max_size = (N + s->R - 1) / s->R;
        unsigned passes = (unsigned)(max_size / d.G + 2);
        unsigned threads = ((d.G + 31) / 32) * 32;
        if (threads > 256) threads = 256;
        draw_direct_reuse_kernel<<<dim3(passes, s->R, batches), threads, 0, st>>>(v, p, off_cur, off_next, N, batches, localize,
                                                                                 s->negs_buf, s->req_keys, s->req_cap);
    } else {
        draw_direct_iid_kernel<<<dim3(grid_for(N, 256), batches), 256, 0, st>>>(v, p, off_cur, off_next, N, batches,
                                                                              d.level == NUPS_NONCONFORM, localize,
                                                                              s->negs_buf, s->req_keys, s->req_cap);
    }
    LAUNCH_CHECK(s);
    d.cur ^= 1;
    if (localize) {
        rc = nups_localize_apply(s, N, st);
        if (rc != NUPS_OK) return rc;
    }
    s->last_negs_n = N;
    if (batches > 1) {
        s->ahead_dist = dist; s->ahead_N = N; s->ahead_total = batches; s->ahead_next = 1;
    }
    return NUPS_OK;
}

extern "C" nups_status nups_last_negatives(nups_store* s, const uint32_t** h_d_keys_out, uint64_t* h_n_out)
{
    if (!s || !h_d_keys_out || !h_n_out) return NUPS_EINVAL;
    *h_d_keys_out = s->last_negs;
    *h_n_out = s->last_negs_n;
    return NUPS_OK;
}
