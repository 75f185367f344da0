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
    if ((level == NUPS_LONGTERM || level == NUPS_NONCONFORM) && !s->own) return NUPS_ESTATE;
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
        rc = nups_dev_alloc(s, &d.table, n * sizeof(AliasEntry));
        if (rc != NUPS_OK) return rc;
        unsigned g = grid_for(n, 256);
        alias_classify_kernel<<<g, 256, 0, st>>>(d_weights, n, W, lrank, dex, sex);
        LAUNCH_CHECK(s);
        rc = nups_scan_u64(s, lrank, lrank, n, d_nL, sc, st);
        if (rc == NUPS_OK) rc = nups_scan_u64(s, dex, dex, n, nullptr, sc, st);
        if (rc == NUPS_OK) rc = nups_scan_u64(s, sex, sex, n, nullptr, sc, st);
        if (rc != NUPS_OK) { nups_dev_free(s, d.table, n * sizeof(AliasEntry)); return rc; }
        unsigned long long nL = 0;
        CK(cudaMemcpyAsync(&nL, d_nL, 8, cudaMemcpyDeviceToHost, st));
        CK(cudaStreamSynchronize(st));
        alias_rank_kernel<<<g, 256, 0, st>>>(d_weights, n, W, lrank, dex, sex, nL, inc, hidx);
        LAUNCH_CHECK(s);
        alias_fill_kernel<<<g, 256, 0, st>>>(d_weights, n, W, lrank, dex, nL, inc, hidx, (AliasEntry*)d.table);
        LAUNCH_CHECK(s);
        CK(cudaStreamSynchronize(st));
    }
    if (nups_dev_alloc(s, (void**)&d.off, 2 * s->R * 8) != NUPS_OK) {
        nups_dev_free(s, d.table, d.table ? n * sizeof(AliasEntry) : 0);
        return NUPS_ENOMEM;
    }
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

// Handle buffer layout (device): keys[N] (u32) | post[N] (u32) | state[3][R] (uint4) | flags | prefix
struct HandleView {
    uint32_t* keys;
    uint32_t* post;    // LONG-TERM: postponed entries of each sub-handle, in the order they were postponed
    uint4* state;      // LONG-TERM per sub-handle: x = walk position, y = postponed head, z = postponed tail
    uint4* prev;       //   the state before the running call
    uint4* walk;       //   what the running call does: x = fresh entries walked, y = of those local,
                       //   z = postponed entries emitted
    uint32_t* flags;   // LONG-TERM: "is local" bit of every fresh entry, and the number of local entries before
    uint32_t* prefix;  //   each 32-entry word; sub-handle q owns the words from (b_q / 32) + q on
};
static size_t handle_bytes(uint64_t N, uint32_t R, int level)
{
    size_t b = align256(N * 4);
    if (level == NUPS_LONGTERM) b += align256(N * 4) + 3 * align256((size_t)R * 16) + 2 * align256((N / 32 + R + 2) * 4);
    return b;
}
static HandleView handle_view(char* buf, uint64_t N, uint32_t R, int level)
{
    HandleView h;
    memset(&h, 0, sizeof(h));
    h.keys = (uint32_t*)buf; buf += align256(N * 4);
    if (level == NUPS_LONGTERM) {
        h.post = (uint32_t*)buf; buf += align256(N * 4);
        h.state = (uint4*)buf; buf += align256((size_t)R * 16);
        h.prev = (uint4*)buf; buf += align256((size_t)R * 16);
        h.walk = (uint4*)buf; buf += align256((size_t)R * 16);
        h.flags = (uint32_t*)buf; buf += align256((N / 32 + R + 2) * 4);
        h.prefix = (uint32_t*)buf; buf += align256((N / 32 + R + 2) * 4);
    }
    return h;
}

// Local sampling: the first key local to worker q among the candidate k0 and the 63 keys after it
// (wrapping inside the distribution's key range), else k0.  The candidates are consecutive keys, so
// their ownership words are consecutive too.  Four lanes serve one candidate: each reads the four words
// of its part of a 16-key group with one 128-bit load (the four loads of a candidate fall into one cache
// line, so a warp instruction touches 8 lines instead of 32), and the walk goes group by group until
// a local key shows up (most walks end within the first group).
// Called by all four lanes of a quad with the same arguments; whole warps must call.
__device__ __forceinline__ uint32_t first_local_quad(const View& v, const DrawParams& p, uint32_t q, uint32_t k0,
                                                     bool active)
{
    const unsigned sub = threadIdx.x & 3;
    const uint32_t R = v.R;
    uint32_t result = k0;
    bool searching = active && v.own != nullptr;
    const unsigned long long rel = k0 - p.key_base;
    const uint32_t a0 = k0 & ~3u;                            // 16-byte aligned start
    if (searching && !(rel + NUPS_LOCAL_PROBES <= p.n && (uint64_t)a0 + NUPS_LOCAL_PROBES + 16 <= v.num_keys)) {
        // near the end of the key range: probe one key at a time
        for (uint32_t probe = 0; probe < NUPS_LOCAL_PROBES; ++probe) {
            const uint32_t cand = p.key_base + (uint32_t)((rel + probe) % p.n);
            if (key_is_local(v, q, cand)) { result = cand; break; }
        }
        searching = false;
    }
    const uint32_t res0 = searching ? a0 % R : 0u;           // key mod R of key a0
    for (uint32_t g = 0; g < NUPS_LOCAL_PROBES / 16 + 1; ++g) {
        if (!__any_sync(0xFFFFFFFFu, searching)) break;
        uint32_t m = 0;                                      // bit t: my key t is a candidate and local
        const uint32_t kb = a0 + 16 * g + 4 * sub;           // my four keys: kb ... kb + 3
        if (searching) {
            const uint4 o = __ldg(reinterpret_cast<const uint4*>(v.own + kb));
            const uint32_t hw = v.H ? __ldg(v.hot_bits + (kb >> 5)) >> (kb & 31) : 0u;     // replicated: local to all
            uint32_t r = (res0 + 16 * g + 4 * sub) % R;
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const uint32_t w = t == 0 ? o.x : t == 1 ? o.y : t == 2 ? o.z : o.w;
                const uint32_t ob = w & 0xFFu;
                const bool loc = (ob == NUPS_OWNER_DEFAULT ? r : ob) == q || ((hw >> t) & 1u);
                const uint32_t key = kb + t;
                if (loc && key >= k0 && key - k0 < NUPS_LOCAL_PROBES) m |= 1u << t;
                r = r + 1 == R ? 0u : r + 1;
            }
            m <<= 4 * sub;
        }
        m |= __shfl_xor_sync(0xFFFFFFFFu, m, 1);
        m |= __shfl_xor_sync(0xFFFFFFFFu, m, 2);
        if (searching && m) {
            result = a0 + 16 * g + (uint32_t)(__ffs(m) - 1);
            searching = false;
        }
    }
    return result;
}

// one candidate per lane: the quads take the warp's candidates eight at a time
__device__ __forceinline__ uint32_t first_local_warp(const View& v, const DrawParams& p, uint32_t q, uint32_t k0,
                                                     bool active)
{
    const unsigned lane = threadIdx.x & 31;
    uint32_t mine = k0;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int src = 8 * r + (int)(lane >> 2);
        const uint32_t kk = __shfl_sync(0xFFFFFFFFu, k0, src);
        const uint32_t qq = __shfl_sync(0xFFFFFFFFu, q, src);
        const bool act = __shfl_sync(0xFFFFFFFFu, (int)active, src) != 0;
        const uint32_t res = first_local_quad(v, p, qq, kk, act);
        const uint32_t back = __shfl_sync(0xFFFFFFFFu, res, 4 * (int)(lane & 7));
        if ((int)(lane >> 3) == r) mine = back;
    }
    return mine;
}

// independent draws: one thread per sample.  The advanced stream offsets go to the other half of the
// distribution's offset array.
__global__ void draw_iid_kernel(View v, DrawParams p, const unsigned long long* __restrict__ off_cur,
                                unsigned long long* __restrict__ off_next, HandleView h, uint64_t N, int localize)
{
    grid_dependency_wait();
    const uint32_t R = v.R;
    if (blockIdx.x == 0)
        for (uint32_t w = threadIdx.x; w < R; w += blockDim.x)
            off_next[w] = off_cur[w] + (chunk_begin(w + 1, N, R) - chunk_begin(w, N, R));
    uint64_t o = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (o >= N) return;
    const uint32_t q = chunk_of_pos(o, N, R);
    const uint32_t k = draw_iid(p, q, off_cur[q] + (o - chunk_begin(q, N, R)));
    h.keys[o] = k;
    if (localize)                                  // PrepareSample localizes what it sampled
        mark_localize_rare(v, k, q, __popc(__match_any_sync(__activemask(), k)) > 1);
}

// Pooled reuse: pool `pl` of a worker holds G iid draws and is walked U times, each pass in a fresh
// Fisher-Yates order.  Stream position s lies in pass number s / G overall (pool = pass / U).
// One block visits one pool: it draws the pool once, then shuffles up to T passes at a time.  A shuffle
// is a chain of dependent swaps, so each of the T passes gets one thread, and the passes' arrays are
// interleaved ([element][pass]) so that the threads of a warp work side by side in shared memory;
// drawing the swap partners and writing the output are block-wide.
// Shared memory: pool[G] (u32) | partner[G][T] (u16) | perm[G][T] (u16).
constexpr unsigned REUSE_THREADS = 512;
struct ReuseShape {
    unsigned T;
    size_t smem;
};
static ReuseShape reuse_shape(uint32_t U, uint32_t G)
{
    ReuseShape r;
    r.T = U < 32 ? U : 32;
    while (r.T > 1 && (size_t)r.T * G * 4 > 40 * 1024) r.T--;
    r.smem = (size_t)G * 4 + (size_t)r.T * G * 4;
    return r;
}
static unsigned reuse_pools(uint64_t max_size, uint32_t U, uint32_t G)
{
    return (unsigned)(max_size / ((uint64_t)U * G) + 2);      // a stretch may begin and end inside a pool
}

// emit(in, key, position in the stretch, mark): called by whole warps for every output position; `mark` says
// whether the key still has to be localized there.  When a whole pass of the pool lies inside the stretch, every
// key of the pool is sampled by this call, so the pool's keys are localized once each (mark_key) instead of once
// per output position (U times as often).
template <class Emit, class Mark>
__device__ __forceinline__ void reuse_pool_visit(const DrawParams& p, uint32_t q, unsigned long long s0,
                                                 unsigned long long s1, uint32_t T, Emit emit, Mark mark_key)
{
    extern __shared__ __align__(16) uint32_t reuse_mem[];
    const uint32_t G = p.G, U = p.U;
    const unsigned tid = threadIdx.x;
    const unsigned long long span = (unsigned long long)U * G;
    const unsigned long long pl = s0 / span + blockIdx.x;
    if (pl * span >= s1) return;
    uint32_t* pool = reuse_mem;
    uint16_t* partner = reinterpret_cast<uint16_t*>(reuse_mem + G);
    uint16_t* perm = partner + (size_t)T * G;
    bool whole_pass;                                         // does a pass of this pool lie fully inside [s0, s1)?
    {
        const unsigned long long first = (s0 + G - 1) / G, last_plus_1 = s1 / G;           // passes fully inside
        const unsigned long long lo = first > pl * U ? first : pl * U;
        const unsigned long long hi = last_plus_1 < (pl + 1) * U ? last_plus_1 : (pl + 1) * U;
        whole_pass = lo < hi;
    }
    for (uint32_t m = tid; m < G; m += blockDim.x) {
        const uint32_t k = draw_iid(p, q, pl * G + m);
        pool[m] = k;
        if (whole_pass) mark_key(k);
    }
    const uint32_t blocks_per_pass = (G + 2) / 4;            // Philox blocks that hold the G - 1 shuffle words
    for (uint32_t t0 = 0; t0 < U; t0 += T) {
        const uint32_t nt = U - t0 < T ? U - t0 : T;
        const unsigned long long pass0 = pl * U + t0;
        if ((pass0 + nt) * G <= s0 || pass0 * G >= s1) continue;          // none of these passes is asked for
        __syncthreads();
        // swap partners: step i = G-1 ... 1 of a pass swaps i with mulhi(x, i + 1), x = word G-1-i of the
        // pass's Philox stream (purpose 1, four words per block)
        for (uint32_t e = tid; e < nt * blocks_per_pass; e += blockDim.x) {
            const uint32_t t = e / blocks_per_pass, blk = e % blocks_per_pass;
            uint32_t x[4];
            philox_at(p.seed, pass0 + t, q, 1, blk, x);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t d = blk * 4 + k;
                if (d + 1 < G) partner[(size_t)(G - 1 - d) * T + t] = (uint16_t)__umulhi(x[k], G - d);
            }
        }
        for (uint32_t e = tid; e < nt * G; e += blockDim.x) perm[(size_t)(e / nt) * T + e % nt] = (uint16_t)(e / nt);
        __syncthreads();
        if (tid < nt) {
            // the swaps depend on one another; their partners do not and are fetched eight at a time
            uint16_t* pm = perm + tid;
            const uint16_t* pa = partner + tid;
            uint32_t i = G - 1;
            for (; i >= 8; i -= 8) {
                uint32_t r[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) r[k] = pa[(size_t)(i - k) * T];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint16_t tmp = pm[(size_t)(i - k) * T];
                    pm[(size_t)(i - k) * T] = pm[(size_t)r[k] * T];
                    pm[(size_t)r[k] * T] = tmp;
                }
            }
            for (; i >= 1; --i) {
                const uint32_t r = pa[(size_t)i * T];
                const uint16_t tmp = pm[(size_t)i * T]; pm[(size_t)i * T] = pm[(size_t)r * T]; pm[(size_t)r * T] = tmp;
            }
        }
        __syncthreads();
        const uint32_t total = nt * G;
        for (uint32_t e0 = 0; e0 < total; e0 += blockDim.x) {          // whole warps: emit may ballot
            const uint32_t e = e0 + tid;
            const uint32_t t = e / G, j = e % G;
            const unsigned long long sp = (pass0 + t) * G + j;
            const bool in = e < total && sp >= s0 && sp < s1;
            const uint32_t k = in ? pool[perm[(size_t)j * T + t]] : 0u;
            emit(in, k, sp - s0, !whole_pass);
        }
    }
}

__global__ void draw_reuse_kernel(View v, DrawParams p, const unsigned long long* __restrict__ off_cur,
                                  unsigned long long* __restrict__ off_next, HandleView h, uint64_t N, int localize,
                                  int longterm, uint32_t T)
{
    grid_dependency_wait();
    const uint32_t q = blockIdx.y, R = v.R;
    const unsigned long long b0 = chunk_begin(q, N, R), size = chunk_begin(q + 1, N, R) - b0;
    const unsigned long long s0 = off_cur[q];
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        off_next[q] = s0 + size;
        if (longterm) h.state[q] = make_uint4(0u, 0u, 0u, 0u);
    }
    if (size == 0) return;
    reuse_pool_visit(p, q, s0, s0 + size, T, [&](bool in, uint32_t k, unsigned long long rel, bool mark) {
        if (in) {
            h.keys[b0 + rel] = k;
            if (localize && mark) mark_localize(v, k, q);
        }
    }, [&](uint32_t k) { if (localize) mark_localize(v, k, q); });
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
        size_t want = need + need / 4;
        if (s->dev_cap && (want > s->dev_cap || s->dev_bytes - h.cap > s->dev_cap - want)) return NUPS_ENOMEM;
        nups_dev_free(s, h.buf, h.cap);
        h.buf = nullptr; h.cap = 0;
        nups_status rc = nups_dev_alloc(s, (void**)&h.buf, want);
        if (rc != NUPS_OK) return rc;
        h.cap = want;
    }
    const bool reuse = d.level == NUPS_BOUNDED || d.level == NUPS_LONGTERM;
    const bool loc = s->own && d.level != NUPS_NONCONFORM;
    if (loc) {
        nups_status rc = nups_new_epoch(s, st);
        if (rc != NUPS_OK) return rc;
    }
    HandleView hv = handle_view(h.buf, N, s->R, d.level);
    DrawParams p = draw_params(d);
    View v = nups_view(s);
    const unsigned long long* off_cur = d.off + (size_t)d.cur * s->R;
    unsigned long long* off_next = d.off + (size_t)(d.cur ^ 1) * s->R;
    nups_time_begin(s, st, NUPS_TIMED_DRAW);
    if (reuse) {
        const ReuseShape sh = reuse_shape(d.U, d.G);
        nups_launch_dependent(draw_reuse_kernel, dim3(reuse_pools((N + s->R - 1) / s->R, d.U, d.G), s->R), REUSE_THREADS,
                              sh.smem, st, v, p, off_cur, off_next, hv, N, loc, d.level == NUPS_LONGTERM, sh.T);
    } else {
        nups_launch_dependent(draw_iid_kernel, grid_for(N, 256), 256, 0, st, v, p, off_cur, off_next, hv, N, loc);
    }
    nups_time_end(s, st);
    LAUNCH_CHECK(s);
    d.cur ^= 1;
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
    grid_dependency_wait();
    uint64_t o = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    bool in = o < n;
    uint32_t k = 0;
    uint32_t q = 0;
    if (in) {
        k = h.keys[cursor + o];
        if (local_only) q = chunk_of_pos(cursor + o, N, v.R);
    }
    if (local_only) k = first_local_warp(v, p, q, k, in);
    if (in) out[o] = k;
    count_sample(v, k, in);
}

// Reuse with postponing.  Entries of a sub-handle not yet postponed are taken in list order: a local
// one is emitted, a non-local one is re-localized and appended to the sub-handle's postponed queue;
// the walk stops right after the last entry it must emit, and when the fresh entries run out the
// postponed ones are emitted.  Locality is judged by the ownership at the start of the call.
// Where an entry goes depends only on how many local entries lie before it, so the walk is a
// prefix sum, not a loop: (1) one bit per fresh entry, looked up by the whole GPU; (2) per sub-handle,
// a scan of the bit counts that also finds where the walk stops (and emits entries that earlier calls
// postponed); (3) every entry is placed on its own, and what is postponed moves to its worker.
struct LtChunk {
    uint32_t q;
    uint64_t b0, size, take, out_base;
    bool active;
};
__device__ __forceinline__ LtChunk lt_chunk(uint32_t q, uint64_t N, uint32_t R, uint64_t cursor, uint64_t n)
{
    LtChunk c;
    c.q = q;
    c.b0 = chunk_begin(q, N, R);
    const uint64_t b1 = chunk_begin(q + 1, N, R);
    const uint64_t lo = max(c.b0, cursor), hi = min(b1, cursor + n);
    c.active = lo < hi;
    c.size = b1 - c.b0;
    c.take = c.active ? hi - lo : 0;
    c.out_base = c.active ? lo - cursor : 0;
    return c;
}

__global__ void lt_flags_kernel(View v, HandleView h, uint64_t N, uint64_t cursor, uint64_t n, uint32_t q_first)
{
    grid_dependency_wait();
    const LtChunk c = lt_chunk(q_first + blockIdx.y, N, v.R, cursor, n);
    if (!c.active) return;
    const unsigned lane = threadIdx.x & 31;
    const uint64_t oc = h.state[c.q].x;
    const uint64_t word = (oc >> 5) + (((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    if (word * 32 >= c.size) return;
    const uint64_t i = word * 32 + lane;
    const bool loc = i >= oc && i < c.size && key_is_local(v, c.q, h.keys[c.b0 + i]);
    const unsigned bits = __ballot_sync(0xFFFFFFFFu, loc);
    if (lane == 0) h.flags[(c.b0 >> 5) + c.q + word] = bits;
}

constexpr int LT_THREADS = 1024;
constexpr int LT_WORDS = 4;                  // flag words per thread and round of the scan

__global__ void __launch_bounds__(LT_THREADS)
lt_scan_kernel(View v, HandleView h, uint64_t N, uint64_t cursor, uint64_t n, uint32_t q_first,
               uint32_t* __restrict__ out)
{
    grid_dependency_wait();
    __shared__ unsigned sh_tl, sh_old;
    __shared__ unsigned warp_tot[LT_THREADS / 32];
    __shared__ unsigned long long sh_stop;       // walk position right after the last entry that must be emitted
    const LtChunk c = lt_chunk(q_first + blockIdx.x, N, v.R, cursor, n);
    if (!c.active) return;
    const unsigned tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint4 stt = h.state[c.q];
    const uint64_t oc = stt.x, ph = stt.y, pt = stt.z;
    const uint64_t w0 = oc >> 5, w1 = oc < c.size ? (c.size + 31) >> 5 : w0;
    const uint32_t* flags = h.flags + (c.b0 >> 5) + c.q;
    uint32_t* prefix = h.prefix + (c.b0 >> 5) + c.q;
    if (tid == 0) sh_stop = ~0ull;
    unsigned long long carry = 0;                // local entries before the round
    for (uint64_t base = w0; base < w1 && carry < c.take; base += (uint64_t)LT_THREADS * LT_WORDS) {
        uint32_t bits[LT_WORDS];
        unsigned mine = 0;
#pragma unroll
        for (int k = 0; k < LT_WORDS; ++k) {
            const uint64_t w = base + (uint64_t)tid * LT_WORDS + k;
            bits[k] = w < w1 ? flags[w] : 0u;
            mine += __popc(bits[k]);
        }
        unsigned inc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
            if (lane >= (unsigned)o) inc += y;
        }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        unsigned long long before = carry + (inc - mine);
        unsigned total = 0;
        for (unsigned w = 0; w < LT_THREADS / 32; ++w) {
            if (w < warp) before += warp_tot[w];
            total += warp_tot[w];
        }
#pragma unroll
        for (int k = 0; k < LT_WORDS; ++k) {
            const uint64_t w = base + (uint64_t)tid * LT_WORDS + k;
            if (w < w1) prefix[w] = (uint32_t)before;
            const unsigned cnt = __popc(bits[k]);
            if (before < c.take && c.take <= before + cnt) {
                // the take-th local entry is the (take - before)-th set bit of this word
                uint32_t b = bits[k];
                for (unsigned long long skip = c.take - before - 1; skip; --skip) b &= b - 1;
                sh_stop = w * 32 + (unsigned)(__ffs(b) - 1) + 1;
            }
            before += cnt;
        }
        carry += total;
        __syncthreads();
    }
    __syncthreads();
    if (tid == 0) {
        const uint64_t fresh = oc < c.size ? c.size - oc : 0;
        const uint64_t tc = carry >= c.take ? (uint64_t)sh_stop - oc : fresh;      // fresh entries walked
        const uint64_t tl = carry >= c.take ? c.take : (uint64_t)carry;             // of those local = emitted
        const uint64_t cnt = c.take - tl;                                           // postponed entries emitted
        h.prev[c.q] = stt;
        h.walk[c.q] = make_uint4((unsigned)tc, (unsigned)tl, (unsigned)cnt, 0u);
        h.state[c.q] = make_uint4((unsigned)(oc + tc), (unsigned)(ph + cnt), (unsigned)(pt + tc - tl), 0u);
        sh_tl = (unsigned)tl;
        sh_old = (unsigned)(cnt < pt - ph ? cnt : pt - ph);         // postponed by earlier calls, emitted by this one
    }
    __syncthreads();
    // postponed entries come after the local ones; those that earlier calls postponed are already in place
    // (what this call postpones and emits is handled where it is placed)
    const unsigned tl = sh_tl, old = sh_old;
    for (unsigned j0 = 0; j0 < old; j0 += LT_THREADS) {
        const unsigned j = j0 + tid;
        const bool in = j < old;
        uint32_t key = 0;
        if (in) {
            key = h.post[c.b0 + ph + j];
            out[c.out_base + tl + j] = key;
        }
        count_sample(v, key, in);
    }
}

// C8 > 0: the kernel also copies the rows of the keys it emits (rows of C8 chunks of 32 bytes, 32 / C8 rows per warp
// instruction, as gather8_kernel does), which saves the separate gather launch of a full PullSample with values.
template <int C8>
__global__ void __launch_bounds__(256)
lt_place_kernel(View v, HandleView h, uint64_t N, uint64_t cursor, uint64_t n, uint32_t q_first,
                uint32_t* __restrict__ out, const float* __restrict__ table, const float* slab,
                float* __restrict__ out_vals)
{
    grid_dependency_wait();
    const LtChunk c = lt_chunk(q_first + blockIdx.y, N, v.R, cursor, n);
    if (!c.active) return;
    const unsigned lane = threadIdx.x & 31;
    const uint4 pv = h.prev[c.q], wk = h.walk[c.q];
    const uint64_t oc = pv.x, ph = pv.y, pt = pv.z, end = oc + wk.x, tl = wk.y, cnt = wk.z;
    const uint64_t word = (oc >> 5) + (((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    if (word * 32 >= end) return;
    const uint64_t i = word * 32 + lane;
    const bool walked = i >= oc && i < end;
    const uint32_t bits = h.flags[(c.b0 >> 5) + c.q + word];
    const uint64_t before = (uint64_t)h.prefix[(c.b0 >> 5) + c.q + word] + __popc(bits & ((1u << lane) - 1u));
    const bool loc = (bits >> lane) & 1u;
    uint32_t key = 0;
    bool emitted = false;
    uint32_t opos = 0;                                               // where the emitted key went
    if (walked) {
        key = h.keys[c.b0 + i];
        if (loc) {
            opos = (uint32_t)(c.out_base + before);
            out[opos] = key;
            emitted = true;
        } else {
            // postponed: queued behind the non-local entries before it, emitted by this very call if the queue's
            // head gets that far, and moved to the worker.  (Locality was judged before any key moved: the bits
            // were all looked up by the kernel before this one.)
            const uint64_t at = pt + ((i - oc) - before);
            h.post[c.b0 + at] = key;
            if (at >= ph && at < ph + cnt) {
                opos = (uint32_t)(c.out_base + tl + (at - ph));
                out[opos] = key;
                emitted = true;
            }
            mark_localize(v, key, c.q);
        }
    }
    count_sample(v, key, emitted);
    if (C8 > 0) {
        constexpr int RPI = C8 > 0 ? 32 / C8 : 1, UNR = 2;
        const unsigned sub = lane / (C8 > 0 ? C8 : 1), ch = lane % (C8 > 0 ? C8 : 1);
        const uint64_t L = (uint64_t)v.L4 * 4;
        const uint32_t src = emitted ? key : 0xFFFFFFFFu;
        uint32_t pend = 0xFFFFFFFFu;                                 // replica row of a replicated key
        if (emitted && key_is_hot(v, key)) pend = c.q * (uint32_t)v.Hcap + (uint32_t)__ldg(v.slot_of + key);
        for (int r0 = 0; r0 < 32; r0 += UNR * RPI) {
            uint32_t so[UNR], po[UNR], oo[UNR];
            F8 a[UNR];
#pragma unroll
            for (int u = 0; u < UNR; ++u) {
                const int row = r0 + u * RPI + (int)sub;
                so[u] = __shfl_sync(0xFFFFFFFFu, src, row);
                po[u] = __shfl_sync(0xFFFFFFFFu, pend, row);
                oo[u] = __shfl_sync(0xFFFFFFFFu, opos, row);
            }
#pragma unroll
            for (int u = 0; u < UNR; ++u) {
                if (so[u] == 0xFFFFFFFFu) continue;
                const float* p = table + (uint64_t)so[u] * L + 8 * ch;
                a[u] = po[u] == 0xFFFFFFFFu ? ld8_stream(p) : ld8_cached(p);
                if (po[u] != 0xFFFFFFFFu) {
                    const F8 d = ld8_plain(slab + (uint64_t)po[u] * L + 8 * ch);
                    a[u].a = add4(a[u].a, d.a);
                    a[u].b = add4(a[u].b, d.b);
                }
            }
#pragma unroll
            for (int u = 0; u < UNR; ++u)
                if (so[u] != 0xFFFFFFFFu) st8_stream(out_vals + (uint64_t)oo[u] * L + 8 * ch, a[u]);
        }
    }
}

static nups_status pull_internal(nups_store* s, int id, uint64_t n, uint32_t* d_keys_out, float* d_vals_out,
                                 cudaStream_t st)
{
    Handle& h = s->handle[id];
    Dist& d = s->dist[h.dist];
    if (n > h.N - h.cursor) return NUPS_ESTATE;
    if (n == 0) return NUPS_OK;
    if (d.level == NUPS_LONGTERM) {
        nups_status rc = nups_new_epoch(s, st);
        if (rc != NUPS_OK) return rc;
    }
    View v = nups_view(s);
    HandleView hv = handle_view(h.buf, h.N, s->R, d.level);
    DrawParams p = draw_params(d);
    if (d.level == NUPS_LONGTERM) {
        // sub-handles overlapped by [cursor, cursor + n)
        uint32_t qf = 0, ql = 0;
        for (uint32_t q = 0; q < s->R; ++q) {
            uint64_t b0 = ((uint64_t)q * h.N) / s->R, b1 = ((uint64_t)(q + 1) * h.N) / s->R;
            if (b0 <= h.cursor && h.cursor < b1) qf = q;
            if (b0 <= h.cursor + n - 1 && h.cursor + n - 1 < b1) ql = q;
        }
        const uint64_t max_size = (h.N + s->R - 1) / s->R;
        const dim3 by_word(grid_for(max_size / 32 + 2, 8), ql - qf + 1);
        nups_launch_dependent(lt_flags_kernel, by_word, 256, 0, st, v, hv, h.N, h.cursor, n, qf);
        LAUNCH_CHECK(s);
        nups_launch_dependent(lt_scan_kernel, ql - qf + 1, LT_THREADS, 0, st, v, hv, h.N, h.cursor, n, qf, d_keys_out);
        LAUNCH_CHECK(s);
        // a full pull of a fresh handle has no entries postponed by earlier calls to emit: the placement pass can copy
        // the rows itself (one table of 64, 128 or 256 floats per row, 32-byte aligned output)
        const uint32_t c8 = s->L / 8;
        const bool fused = d_vals_out && s->vb == 4 && h.cursor == 0 && n == h.N && s->L % 8 == 0 && (c8 == 8 || c8 == 16 || c8 == 32) &&
                           ((uintptr_t)d_vals_out & 31) == 0 && (uint64_t)s->R * s->Hcap < 0xFFFFFFFFull;
        if (fused) nups_time_begin(s, st, NUPS_TIMED_SAMPLE_ROWS);
        if (fused && c8 == 8) nups_launch_dependent(lt_place_kernel<8>, by_word, 256, 0, st, v, hv, h.N, h.cursor, n, qf, d_keys_out, s->val, s->dval, d_vals_out);
        else if (fused && c8 == 16) nups_launch_dependent(lt_place_kernel<16>, by_word, 256, 0, st, v, hv, h.N, h.cursor, n, qf, d_keys_out, s->val, s->dval, d_vals_out);
        else if (fused) nups_launch_dependent(lt_place_kernel<32>, by_word, 256, 0, st, v, hv, h.N, h.cursor, n, qf, d_keys_out, s->val, s->dval, d_vals_out);
        else nups_launch_dependent(lt_place_kernel<0>, by_word, 256, 0, st, v, hv, h.N, h.cursor, n, qf, d_keys_out, nullptr, nullptr, nullptr);
        if (fused) nups_time_end(s, st);
        LAUNCH_CHECK(s);
        if (fused) {
            h.cursor += n;
            h.used = 0;
            return NUPS_OK;
        }
    } else if (d_vals_out && d.level != NUPS_NONCONFORM && !s->cfg.count_accesses) {
        // keys fixed at PrepareSample and nothing to count: the row gather reads them from the handle and hands them out
        // on its way, which saves a launch
        h.cursor += n;
        if (h.cursor == h.N) h.used = 0;
        return nups_gather_internal(s, hv.keys + (h.cursor - n), n, d_vals_out, nullptr, 1, h.cursor - n, h.N, 0, st, d_keys_out);
    } else {
        nups_launch_dependent(emit_kernel, grid_for(n, 256), 256, 0, st, v, p, hv, h.N, h.cursor, n, d.level == NUPS_NONCONFORM, d_keys_out);
        LAUNCH_CHECK(s);
    }
    if (d_vals_out) {
        nups_status rc = nups_gather_internal(s, d_keys_out, n, d_vals_out, nullptr, 1, h.cursor, h.N, 0, st, nullptr);
        if (rc != NUPS_OK) return rc;
    }
    h.cursor += n;
    if (h.cursor == h.N) h.used = 0;       // released; the buffer stays for the next handle
    return NUPS_OK;
}

extern "C" nups_status nups_pull_sample(nups_store* s, nups_handle handle, uint64_t n, uint32_t* d_keys_out,
                                        void* d_vals_out, void* stream)
{
    if (!s || handle < 0 || handle >= NUPS_MAX_HANDLES || !s->handle[handle].used) return NUPS_EINVAL;
    if (n && !d_keys_out) return NUPS_EINVAL;
    return pull_internal(s, (int)handle, n, d_keys_out, (float*)d_vals_out, (cudaStream_t)stream);
}

// ---------------------------------------------------------------------------------------------
// PrepareSample + one full PullSample (keys only) in a single launch, for the workload steps: the
// same keys as the handle path gives, written straight to `out`.  Stream offsets are read from one
// half of the distribution's offset array and the advanced offsets written to the other half.
// ---------------------------------------------------------------------------------------------
// blockIdx.y (iid) / blockIdx.z (reuse) = batch: `batches` handles of N samples each are drawn back to back,
// exactly as that many separate calls would draw them; batch b goes to out + b * N.
__global__ void draw_direct_iid_kernel(View v, DrawParams p, const unsigned long long* __restrict__ off_cur,
                                       unsigned long long* __restrict__ off_next, uint64_t N, uint32_t batches,
                                       int local_only, int localize, uint32_t* __restrict__ out)
{
    grid_dependency_wait();
    const uint64_t o = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t bt = blockIdx.y;
    const bool in = o < N;
    uint32_t k = 0, q = 0;
    out += (uint64_t)bt * N;
    if (in) {
        q = chunk_of_pos(o, N, v.R);
        const unsigned long long size = chunk_begin(q + 1, N, v.R) - chunk_begin(q, N, v.R);
        k = draw_iid(p, q, off_cur[q] + (unsigned long long)bt * size + (o - chunk_begin(q, N, v.R)));
    }
    if (local_only) k = first_local_warp(v, p, q, k, in);
    const bool repeats = localize && __popc(__match_any_sync(0xFFFFFFFFu, in ? k : 0xFFFFFFFFu - (threadIdx.x & 31))) > 1;
    if (in) {
        out[o] = k;
        if (localize) mark_localize_rare(v, k, q, repeats);
    }
    count_sample(v, k, in);
    if (blockIdx.x == 0 && blockIdx.y == 0)
        for (uint32_t w = threadIdx.x; w < v.R; w += blockDim.x)
            off_next[w] = off_cur[w] + (unsigned long long)batches * (chunk_begin(w + 1, N, v.R) - chunk_begin(w, N, v.R));
}

__global__ void draw_direct_reuse_kernel(View v, DrawParams p, const unsigned long long* __restrict__ off_cur,
                                         unsigned long long* __restrict__ off_next, uint64_t N, uint32_t batches,
                                         int localize, uint32_t* __restrict__ out, uint32_t T)
{
    grid_dependency_wait();
    const uint32_t q = blockIdx.y, R = v.R;
    if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0)
        for (uint32_t w = threadIdx.x; w < R; w += blockDim.x)
            off_next[w] = off_cur[w] + (unsigned long long)batches * (chunk_begin(w + 1, N, R) - chunk_begin(w, N, R));
    const unsigned long long b0 = chunk_begin(q, N, R), size = chunk_begin(q + 1, N, R) - b0;
    if (size == 0) return;
    out += (uint64_t)blockIdx.z * N;
    const unsigned long long s0 = off_cur[q] + (unsigned long long)blockIdx.z * size;
    reuse_pool_visit(p, q, s0, s0 + size, T, [&](bool in, uint32_t k, unsigned long long rel, bool mark) {
        if (in) {
            out[b0 + rel] = k;
            if (localize && mark) mark_localize(v, k, q);
        }
        count_sample(v, k, in);
    }, [&](uint32_t k) { if (localize) mark_localize(v, k, q); });
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
    const uint32_t batches = (plain && !s->cfg.deterministic && !s->cfg.count_accesses && !s->own &&
                              N * NUPS_SAMPLE_AHEAD < (1ull << 28)) ? NUPS_SAMPLE_AHEAD : 1;
    if (N * batches > s->negs_cap) {
        uint64_t want = N * batches + N / 4;
        if (s->dev_cap && (want * 4 > s->dev_cap || s->dev_bytes - s->negs_cap * 4 > s->dev_cap - want * 4)) return NUPS_ENOMEM;
        nups_dev_free(s, s->negs_buf, s->negs_cap * 4);
        s->negs_buf = nullptr; s->negs_cap = 0;
        rc = nups_dev_alloc(s, (void**)&s->negs_buf, want * 4);
        if (rc != NUPS_OK) return rc;
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
    const int localize = s->own && d.level != NUPS_NONCONFORM;
    if (localize) {
        rc = nups_new_epoch(s, st);
        if (rc != NUPS_OK) return rc;
    }
    View v = nups_view(s);
    DrawParams p = draw_params(d);
    const unsigned long long* off_cur = d.off + (size_t)d.cur * s->R;
    unsigned long long* off_next = d.off + (size_t)(d.cur ^ 1) * s->R;
    if (d.level == NUPS_BOUNDED) {
        const ReuseShape sh = reuse_shape(d.U, d.G);
        nups_launch_dependent(draw_direct_reuse_kernel, dim3(reuse_pools((N + s->R - 1) / s->R, d.U, d.G), s->R, batches),
                              REUSE_THREADS, sh.smem, st, v, p, off_cur, off_next, N, batches, localize, s->negs_buf, sh.T);
    } else {
        nups_launch_dependent(draw_direct_iid_kernel, dim3(grid_for(N, 256), batches), 256, 0, st, v, p, off_cur, off_next, N, batches,
                                                                              d.level == NUPS_NONCONFORM, localize,
                                                                              s->negs_buf);
    }
    LAUNCH_CHECK(s);
    d.cur ^= 1;
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
