// lvlm_merge_compact: P_new = W_v x P_merged and P_compressed = [P_unmerged, P_new]
// (Section 3.2.1, paragraph 4), applied to the hidden states, to that layer's K and V and
// to the position ids.
//
// Launches: (1) a plan kernel, one CTA per sequence, turns `rank` into a source-row map for
// every output row, a destination for every input row and a merge weight for every image token;
// (2) one streaming kernel reads every input row of the hidden states once, moves it if it is
// kept and adds it to the weighted sum if it is merged; (3) one kernel compacts K and V in place.
#include <mutex>

#include "common.cuh"
#include "compact.cuh"
#include "merge.cuh"
#include "sm100.cuh"

namespace lvlm {

struct MergeLayout {
    int r1, r, Nout, V, kvP;
    HiddenGrid grid;
    size_t off_src, off_dst, off_wgt, off_meta, off_partial, off_kvpartial, total;
};

constexpr int kHidThreads = 256;       // consumer threads: thread = 16-byte column group (+256, +512 ...)
constexpr int kStreamThreads = kHidThreads + 64;   // ... plus the warps that issue the bulk loads and stores
constexpr int kHidMaxChunks = 4;       // column groups per thread: rows up to 4 * 256 * 8 = 8192 channels
constexpr int kNoRow = -2147483647 - 1;  // marks a slot of a tile that holds no row
constexpr int kHidCluster = 8;         // CTAs whose partial sums are added through shared memory
constexpr int kMaxHidPartials = 80;    // partial rows of a sequence the launch accepts when it makes the clusters smaller
constexpr int kStreamMaxStages = 16;   // tiles in flight per CTA
constexpr int kStreamRingBytes = 172 * 1024;  // shared-memory ring of a CTA (one CTA per SM)
constexpr int kStreamTileBytes = 34 * 1024;   // rows are grouped into tiles of about this size
constexpr int kKvRowBytes = kHeadDim * 2;

// One CTA per SM over the whole batch, at least two tiles of rows each; the CTAs of a sequence form
// clusters (their partial sums of the merged row are added through distributed shared memory).
HiddenGrid hidden_grid(const lvlm_dims* d) {
    HiddenGrid g;
    g.V = d->C / 8;
    const int rowB = d->C * 2;
    int rpt = kStreamTileBytes / rowB;
    rpt = rpt < 1 ? 1 : (rpt > 32 ? 32 : rpt);
    g.rpt = rpt;
    g.slotB = rpt * rowB;
    if (g.slotB < 16 * kKvRowBytes) g.slotB = 16 * kKvRowBytes;    // room for a tile of K or V rows
    g.slotB = (g.slotB + 127) / 128 * 128;
    int ns = kStreamRingBytes / g.slotB;
    g.nstage = ns > kStreamMaxStages ? kStreamMaxStages : ns;
    const int tiles = (d->N + rpt - 1) / rpt;
    int raw = 148 / d->B;
    raw = raw > tiles / 2 ? tiles / 2 : raw;
    raw = raw < 1 ? 1 : raw;
    g.cl = 1; g.cps = 0;
    for (int cl = kHidCluster; cl >= 1; cl >>= 1) {        // the cluster size that uses the most CTAs, the larger on a tie
        const int c = raw / cl * cl;
        if (c >= 1 && c / cl <= 48 && c > g.cps) { g.cps = c; g.cl = cl; }
    }
    if (g.cps == 0) { g.cps = raw > 48 ? 48 : raw; g.cl = 1; }
    return g;
}

// Chunks the image span of every K and V sequence is cut into when the merged rows are summed: about four
// work items per CTA of the sequence's batch element (the CTAs take them in turn), not shorter than 128 rows.
static int kv_chunks(const lvlm_dims* d, const HiddenGrid& g) {
    if (d->Hkv <= 0) return 1;
    int p = (4 * g.cps + d->Hkv * 2 - 1) / (d->Hkv * 2);
    const int by_rows = d->n / 128;
    p = p > by_rows ? by_rows : p;
    p = p < 1 ? 1 : p;
    while (p > 1 && (int64_t)(p - 1) * ((d->n + p - 1) / p) >= d->n) --p;      // no chunk is empty
    return p;
}

static bool merge_layout(const lvlm_dims* d, MergeLayout* L) {
    if (!d || d->B <= 0 || d->N <= 0 || d->n <= 0 || d->C <= 0 || d->C % 8 || d->i0 < 0 ||
        d->k < 0 || d->k > d->n || (int64_t)d->i0 + d->n > d->N)
        return false;
    L->r1 = d->n - d->k;
    L->r = L->r1 > 0 ? L->r1 - 1 : 0;
    L->Nout = d->N - L->r;
    L->V = d->C / 8;
    L->grid = hidden_grid(d);
    L->kvP = kv_chunks(d, L->grid);
    const int cps = L->grid.cps;
    size_t off = 0;
    L->off_src = off;     off = align_up(off + (size_t)d->B * d->N * 4, 256);
    L->off_dst = off;     off = align_up(off + (size_t)d->B * d->N * 4, 256);
    L->off_wgt = off;     off = align_up(off + (size_t)d->B * d->n * 4, 256);
    L->off_meta = off;    off = align_up(off + (size_t)d->B * kMetaInts * 4, 256);
    // (the launch may settle for smaller clusters than grid.cl, up to kMaxHidPartials partial rows a sequence)
    const int few = cps < kMaxHidPartials ? cps : kMaxHidPartials;
    const int prow = cps / L->grid.cl > few ? cps / L->grid.cl : few;
    L->off_partial = off; off = align_up(off + (size_t)d->B * prow * d->C * 4, 256);
    L->off_kvpartial = off;
    if (d->Hkv > 0) off = align_up(off + (size_t)d->B * d->Hkv * 2 * L->kvP * kHeadDim * 4, 256);
    L->total = off;
    return true;
}

size_t merge_compact_workspace(const lvlm_dims* d) {
    if (d && d->merge_mode == LVLM_W_NEAREST_KEPT) return nearest_kept_workspace(d);
    MergeLayout L;
    return merge_layout(d, &L) ? L.total : 0;
}

__device__ __forceinline__ float block_sum_fixed(float v, float* scratch) {
    // fixed reduction tree: xor shuffles inside a warp, then warp 0 over the warp sums
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = (threadIdx.x < (blockDim.x >> 5)) ? scratch[threadIdx.x] : 0.f;
    if (threadIdx.x < 32) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
        if (threadIdx.x == 0) scratch[32] = t;
    }
    __syncthreads();
    return scratch[32];
}

// Weight of the merged token at place p of the queue (p = 0 most important), normalised.
__device__ __forceinline__ float merge_weight(int mode, int p, int r1, float inv_sum,
                                              const float* __restrict__ w_custom) {
    switch (mode) {
        case LVLM_W_LINEAR_RANK: return (float)(r1 - p) * inv_sum;
        case LVLM_W_GEOMETRIC:   return ldexpf(1.0f, -(p < r1 - 1 ? p + 1 : r1 - 1));
        case LVLM_W_UNIFORM:     return inv_sum;
        default:                 return w_custom[p] * inv_sum;
    }
}

__device__ __forceinline__ uint32_t plan_cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void plan_cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n"
                 "barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ int plan_ld_cluster(const int* my_smem, uint32_t rank) {
    uint32_t local = (uint32_t)__cvta_generic_to_shared(my_smem), remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    int v;
    asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(remote) : "memory");
    return v;
}

// A cluster of P CTAs per sequence (grid (P, B)): source map, destination map, weights, position ids,
// new length.  CTA r takes the r-th run of the image tokens: it counts its kept tokens, learns from the
// lower ranks how many came before, then writes the maps of its run (tile by tile, thread = token,
// coalesced).  The position ids are compacted in place in rounds of P x blockDim output rows: every CTA
// loads its rows of the round, a cluster barrier, then it stores them (a row's source lies at or behind it,
// so nothing a later round needs is overwritten).
__global__ void __launch_bounds__(1024)
merge_plan_kernel(const int32_t* __restrict__ rank, int32_t* pos_ids, int N, int i0, int n, int k,
                  int mode, float inv_sum, const float* __restrict__ w_custom,
                  int32_t* __restrict__ src_map, int32_t* __restrict__ dst_map,
                  float* __restrict__ wgt, int32_t* __restrict__ meta, int32_t* new_len,
                  int32_t* dev_status) {
    __shared__ int scan_scratch[33];
    __shared__ float fsum_scratch[33];
    __shared__ int s_total, s_first_drop, s_merged_tok;
    pdl_enter();
    const int b = blockIdx.y, P = (int)gridDim.x, cr = (int)plan_cluster_rank();
    const int r1 = n - k, r = r1 - 1, Nout = N - r;
    const int32_t* rk = rank + (int64_t)b * n;
    int32_t* src = src_map + (int64_t)b * N;
    int32_t* dst = dst_map + (int64_t)b * N;      // output row of every input row, -1 = merged away
    float* w = wgt + (int64_t)b * n;
    const int chunk = (n + P - 1) / P;
    const int c_lo = min(n, cr * chunk), c_hi = min(n, c_lo + chunk);
    if (threadIdx.x == 0) { s_total = 0; s_first_drop = n; s_merged_tok = -1; }

    if (mode == LVLM_W_CUSTOM) {
        float part = 0.f;
        for (int p = threadIdx.x; p < r1; p += blockDim.x) part += w_custom[p];
        const float tot = block_sum_fixed(part, fsum_scratch);
        inv_sum = 1.0f / tot;
    }
    __syncthreads();

    // kept tokens of my run
    bool bad = false;
    int mine = 0;
    for (int t0 = c_lo; t0 < c_hi; t0 += blockDim.x) {
        const int j = t0 + threadIdx.x;
        const int rj = j < c_hi ? rk[j] : n;
        if (j < c_hi && (rj < 0 || rj >= n)) bad = true;
        mine += j < c_hi && rj < k;
    }
    mine = warp_sum(mine);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(&s_total, mine);
    plan_cluster_barrier();
    int kept_before = 0, kept_all = 0;
    for (int q = 0; q < P; ++q) {
        const int t = plan_ld_cluster(&s_total, q);
        kept_before += q < cr ? t : 0;
        kept_all += t;
    }
    if (kept_all != k) bad = true;

    // the maps of my run
    for (int t0 = c_lo; t0 < c_hi; t0 += blockDim.x) {
        const int j = t0 + threadIdx.x;
        const int rj = j < c_hi ? rk[j] : n;              // past the end: counts as dropped, writes nothing
        const int is_kept = j < c_hi && rj < k;
        int total;
        const int off = kept_before + block_exclusive_scan(is_kept, scan_scratch, &total);
        if (j < c_hi) {
            float wj = 0.f;
            if (is_kept) {
                if (off < k) src[i0 + off] = i0 + j;
                dst[i0 + j] = off < k ? i0 + off : -1;
            } else {
                dst[i0 + j] = -1;
                if (rj == k) s_merged_tok = j;
                int p = rj - k;
                p = p < 0 ? 0 : (p >= r1 ? r1 - 1 : p);
                wj = merge_weight(mode, p, r1, inv_sum, w_custom);
            }
            w[j] = wj;
        }
        int fd = (j < c_hi && !is_kept) ? j : n;           // first dropped token: one atomic per warp
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) fd = min(fd, __shfl_xor_sync(0xFFFFFFFFu, fd, o));
        if ((threadIdx.x & 31) == 0 && fd < n) atomicMin(&s_first_drop, fd);
        kept_before += total;
    }
    // rows outside the image span, shared out over the CTAs
    for (int o = cr * blockDim.x + threadIdx.x; o < Nout; o += P * blockDim.x) {
        if (o < i0) { src[o] = o; dst[o] = o; }
        else if (o == i0 + k) src[o] = -1;
        else if (o > i0 + k) { src[o] = o + r; dst[o + r] = o; }
    }
    if (bad && dev_status) atomicOr(dev_status, LVLM_DEV_BOUNDS);
    plan_cluster_barrier();                               // the maps are complete, every CTA's findings are in place
    int first_drop = n, merged_tok = 0;
    for (int q = 0; q < P; ++q) {
        first_drop = min(first_drop, plan_ld_cluster(&s_first_drop, q));
        const int mt = plan_ld_cluster(&s_merged_tok, q);
        if (mt >= 0) merged_tok = mt;
    }
    if (cr == 0 && threadIdx.x == 0) {
        meta[b * kMetaInts + 0] = i0 + first_drop;       // first row whose content changes
        meta[b * kMetaInts + 1] = 0;                     // ticket counter of the merge blocks
        meta[b * kMetaInts + 2] = merged_tok;
        if (new_len) new_len[b] = Nout;
    }
    if (pos_ids) {
        int32_t* pid = pos_ids + (int64_t)b * N;
        const int pos_new = pid[i0 + merged_tok];         // read before any CTA stores (first store: after a barrier)
        for (int o0 = 0; o0 < Nout; o0 += P * blockDim.x) {
            const int o = o0 + cr * blockDim.x + threadIdx.x;
            int val = 0;
            if (o < Nout) { const int sidx = src[o]; val = sidx >= 0 ? pid[sidx] : pos_new; }
            plan_cluster_barrier();
            if (o < Nout) pid[o] = val;
        }
    }
    plan_cluster_barrier();                               // nobody leaves while its shared memory may still be read
}

__global__ void identity_len_kernel(int32_t* new_len, int B, int N) {
    pdl_enter();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) new_len[b] = N;
}

__device__ __forceinline__ uint32_t hid_cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void hid_cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n"
                 "barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ int hid_ld_cluster_i32(const int* my_smem, uint32_t rank) {
    uint32_t local = (uint32_t)__cvta_generic_to_shared(my_smem), remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    int v;
    asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(remote) : "memory");
    return v;
}
__device__ __forceinline__ float4 hid_ld_cluster_f4(const float* my_smem, uint32_t rank) {
    uint32_t local = (uint32_t)__cvta_generic_to_shared(my_smem), remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote) : "memory");
    return v;
}

// One pass over the rows.  grid (CTAs per sequence, B), clusters of `cl` CTAs along x.  A CTA is eight consumer
// warps, a loader warp and a storer warp around a ring of shared-memory tiles, each guarded by a "full" mbarrier
// (bytes landed) and an "empty" mbarrier (every consumer warp and the storer are done with it).  A tile is a run of
// consecutive rows, fetched by ONE bulk copy (cp.async.bulk; a copy costs the issuing warp about as much whatever
// its size, so they are made large), so each row is read exactly once.
//
// First the tiles of K and V (only with Kc): the image span of every (KV head, K|V) is cut into chunks, a CTA
// takes every grid.x-th chunk; the consumers add the rows that are merged away, times their weights, in row
// order, and leave one fp32 partial row per chunk for the compaction kernel, which adds the chunks in order.
// (Kept rows of these tiles come along unused: fetching 256-byte rows one by one would cost more.)
//
// Then the hidden states: tiles of consecutive INPUT rows are dealt round robin, so that every CTA gets the same
// mix of kept rows (read and written) and merged rows (read only).  Kept rows leave again by bulk copies from
// shared memory to their destination (the storer issues one per run of rows whose destinations are contiguous; no
// register ever holds a row), merged rows are added by the consumers to fp32 sums each thread keeps for its columns
// (its rows in increasing order).  The CTAs of a cluster add their sums in rank order through distributed shared
// memory, each a slice of the columns, and park one partial per cluster; the compaction launch that follows adds
// the partials in cluster order, rounds once to bf16 and writes P_new.
// Without `out` nothing is stored: only merged rows are read.
//
// Destination and weight of every row of a tile travel beside it: the loader copies them (cp.async, 4 bytes each)
// into a table a dozen tiles ahead, so that nobody ever waits for them.
struct StreamArgs {
    const char* hid; char* out; char* scratch;
    int64_t hid_sb, out_sb, scr_sb;                      // bytes
    int rowB, V, N, i0, n, k, cl, rpt, slotB, nstage;
    const int32_t* dst_map; const float* wgt; int32_t* meta; float* partial;
    const char* K; const char* Vc; int64_t kv_sb, kv_sh; // bytes
    int Hkv, kvP, kvL, kvT;
    float* kv_partial;
    int32_t* dev_status;
};

constexpr int kTabTiles = 32;          // tiles whose row tables are held at a time
constexpr int kTabAhead = 12;          // ... and how far ahead of the tile being fetched they are requested
constexpr int kTabRows = 64;           // most rows a tile can hold
constexpr int kLoaderWarp = kHidThreads / 32, kStorerWarp = kLoaderWarp + 1;

__device__ __forceinline__ void cp_async4(void* smem, const void* gmem) {
    const uint32_t sa = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(sa), "l"(gmem) : "memory");
}

template <int CH>
__global__ void __launch_bounds__(kStreamThreads, 1) row_stream_kernel(const StreamArgs a) {
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) uint64_t s_full[kStreamMaxStages];
    __shared__ __align__(8) uint64_t s_empty[kStreamMaxStages];
    __shared__ __align__(8) uint64_t s_tab_ready;           // the tables of the tiles fetched before the wait are in place
    __shared__ int s_tab_d[kTabTiles][kTabRows];            // destination and weight of the rows of a tile
    __shared__ float s_tab_w[kTabTiles][kTabRows];
    __shared__ __align__(16) float s_red[16 * kHeadDim];
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int b = blockIdx.y, cta = blockIdx.x, cps = (int)gridDim.x;
    const int S = a.nstage;
    if (tid == 0) {
        for (int s = 0; s < S; ++s) { sm100::mbar_init(&s_full[s], 1); sm100::mbar_init(&s_empty[s], kHidThreads / 32 + 1); }
        sm100::mbar_init(&s_tab_ready, 1);
        s_abort = 0;
        sm100::fence_barrier_init();
    }
    __syncthreads();
    // The kernel ahead in the stream (the plan) writes the row maps and weights only, and it has itself waited for
    // everything before it: the rows can be fetched while it still runs.  The loader does so for the first lap of
    // the ring before it waits; every other warp waits here.  Nobody lets the next kernel start before it has
    // waited itself: that kernel may then take the plan for complete as soon as it runs.
    if (warp != kLoaderWarp) { pdl_wait(); pdl_launch_dependents(); }

    const int32_t* dst = a.dst_map + (int64_t)b * a.N;
    const float* w = a.wgt ? a.wgt + (int64_t)b * a.n - a.i0 : nullptr;     // indexed by sequence position
    // My tiles: first those of my K/V chunks, then those of the hidden states.  Every role walks them with its own
    // iterator (the loader with two: one runs ahead for the row tables); no division outside the start of a chunk.
    const int nItems = a.K ? a.Hkv * 2 * a.kvP : 0;
    struct Tile { int first, cnt, kv, item_end, item; const char* from; };
    struct TileIt {
        const StreamArgs& a; int b, cta, cps, nItems;
        int item, tb, r1, row; const char* seq;
        __device__ TileIt(const StreamArgs& a_, int b_, int cta_, int cps_, int nItems_)
            : a(a_), b(b_), cta(cta_), cps(cps_), nItems(nItems_), item(cta_ - cps_), tb(0), r1(0), row(cta_ * a_.rpt), seq(nullptr) {}
        __device__ bool next(Tile* t) {
            while (item < nItems) {
                if (tb < r1) {
                    t->first = tb; t->cnt = min(a.kvT, r1 - tb); t->kv = 1; t->item = item;
                    t->from = seq + (int64_t)tb * kKvRowBytes;
                    tb += a.kvT;
                    t->item_end = tb >= r1;
                    return true;
                }
                item += cps;
                if (item < nItems) {
                    const int chunk = item % a.kvP, gw = item / a.kvP;
                    tb = a.i0 + chunk * a.kvL;
                    r1 = min(a.i0 + a.n, tb + a.kvL);
                    seq = ((gw & 1) ? a.Vc : a.K) + (int64_t)b * a.kv_sb + (int64_t)(gw >> 1) * a.kv_sh;
                }
            }
            if (row < a.N) {
                t->first = row; t->cnt = min(a.rpt, a.N - row); t->kv = 0; t->item_end = 0; t->item = 0;
                t->from = a.hid + (int64_t)b * a.hid_sb + (int64_t)row * a.rowB;
                row += cps * a.rpt;
                return true;
            }
            return false;
        }
    };
    volatile int* abort_flag = &s_abort;
    auto wait_on = [&](uint64_t* bar, uint32_t parity) -> bool {
        if (sm100::mbar_wait(bar, parity)) return true;
        *abort_flag = 1;
        if (a.dev_status) atomicOr(a.dev_status, LVLM_DEV_TIMEOUT);
        return false;
    };

    float acc[CH][8];
#pragma unroll
    for (int ci = 0; ci < CH; ++ci)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[ci][e] = 0.f;

    if (warp == kLoaderWarp) {
        // ---- loader ----------------------------------------------------------------------------------------
        TileIt ahead(a, b, cta, cps, nItems), it(a, b, cta, cps, nItems);
        int ja = 0;                                         // tiles whose tables have been requested
        auto request_table = [&]() {                        // destination and weight of the rows of the next tile ahead
            Tile t;
            if (ahead.next(&t)) {
                int* td = s_tab_d[ja & (kTabTiles - 1)];
                float* tw = s_tab_w[ja & (kTabTiles - 1)];
                for (int e = lane; e < t.cnt; e += 32) {
                    const int i = t.first + e;
                    cp_async4(&td[e], dst + i);
                    if (w && i >= a.i0 && i < a.i0 + a.n) cp_async4(&tw[e], w + i);
                }
            }
            ++ja;
            asm volatile("cp.async.commit_group;\n" ::: "memory");
        };
        auto fetch = [&](const Tile& t, int slot, int j) {
            unsigned char* sbase = ring + (size_t)slot * a.slotB;
            const uint32_t rb = t.kv ? (uint32_t)kKvRowBytes : (uint32_t)a.rowB;
            if (t.kv || a.out) {                            // the whole tile in one copy
                if (lane == 0) {
                    sm100::mbar_arrive_expect_tx(&s_full[slot], (uint32_t)t.cnt * rb);
                    sm100::bulk_load(sbase, t.from, (uint32_t)t.cnt * rb, &s_full[slot]);
                }
            } else {                                        // merged rows only (cnt <= 32 here)
                const bool need = lane < t.cnt && s_tab_d[j & (kTabTiles - 1)][lane] == -1;
                const unsigned bal = __ballot_sync(0xFFFFFFFFu, need);
                if (lane == 0) sm100::mbar_arrive_expect_tx(&s_full[slot], (uint32_t)__popc(bal) * rb);
                __syncwarp();
                if (need) sm100::bulk_load(sbase + (size_t)lane * rb, t.from + (int64_t)lane * rb, rb, &s_full[slot]);
            }
        };
        Tile t;
        int slot = 0, j = 0;
        bool more = it.next(&t);
        // whole-tile copies need no table: the first lap of the ring starts before the wait
        for (; more && j < S && (t.kv || a.out); ++j, ++slot) { fetch(t, slot, j); more = it.next(&t); }
        pdl_wait();
        pdl_launch_dependents();
        for (int q = 0; q < j + kTabAhead; ++q) request_table();
        asm volatile("cp.async.wait_group %0;\n" ::"n"(kTabAhead) : "memory");          // the tables of the tiles under way
        __syncwarp();
        if (lane == 0) sm100::mbar_arrive(&s_tab_ready);
        uint32_t phase = 0;                                 // parity of the "empty" phase awaited; no wait in the first lap
        bool ok = true, first_lap = true;
        if (slot == S) { slot = 0; first_lap = false; }
        while (more) {
            request_table();
            if (!first_lap && ok) ok = wait_on(&s_empty[slot], phase);                // everybody is done with the slot
            asm volatile("cp.async.wait_group %0;\n" ::"n"(kTabAhead) : "memory");      // the table of this tile is in place
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (ok) fetch(t, slot, j);
            ++j;
            if (++slot == S) { slot = 0; if (first_lap) first_lap = false; else phase ^= 1u; }
            more = it.next(&t);
        }
        asm volatile("cp.async.wait_group 0;\n" ::: "memory");
    } else if (warp == kStorerWarp) {
        // ---- storer: lane l owns row l of a tile -------------------------------------------------------------
        TileIt it(a, b, cta, cps, nItems);
        Tile t;
        int slot = 0, j = 0, prev_slot = -1;
        uint32_t phase = 0;
        bool ok = wait_on(&s_tab_ready, 0);
        while (it.next(&t)) {
            if (ok) ok = wait_on(&s_full[slot], phase);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (ok && !t.kv && a.out) {                     // the kept rows leave again
                const int dd = lane < t.cnt ? s_tab_d[j & (kTabTiles - 1)][lane] : kNoRow;
                char* to = nullptr;
                if (dd >= 0) to = a.out + (int64_t)b * a.out_sb + (int64_t)dd * a.rowB;
                else if (dd <= -2 && dd != kNoRow && a.scratch)       // a row set aside: scratch row -d-2
                    to = a.scratch + (int64_t)b * a.scr_sb + (int64_t)(-dd - 2) * a.rowB;
                // runs of rows whose destinations follow each other leave in one copy, issued by the run's first lane
                const unsigned long long toi = (unsigned long long)to;
                const unsigned long long prev = __shfl_up_sync(0xFFFFFFFFu, toi, 1);
                const bool head = to != nullptr && (lane == 0 || prev == 0ull || prev + (unsigned long long)a.rowB != toi);
                const unsigned heads = __ballot_sync(0xFFFFFFFFu, head);
                const unsigned valid = __ballot_sync(0xFFFFFFFFu, to != nullptr);
                if (head) {
                    const unsigned above = lane == 31 ? 0u : (~0u << (lane + 1));
                    const unsigned stop = (heads | ~valid) & above;              // the next head, or the next row that stays
                    const int end = stop ? __ffs(stop) - 1 : 32;
                    sm100::bulk_store(to, ring + (size_t)slot * a.slotB + (size_t)lane * a.rowB,
                                      (uint32_t)(end - lane) * (uint32_t)a.rowB);
                }
            }
            sm100::bulk_commit();                           // one group per tile, empty or not
            if (prev_slot >= 0) {
                sm100::bulk_wait_read<1>();                 // the stores of the tile before have left its slot
                __syncwarp();
                if (lane == 0) sm100::mbar_arrive(&s_empty[prev_slot]);
            }
            prev_slot = slot;
            ++j;
            if (++slot == S) { slot = 0; phase ^= 1u; }
        }
        sm100::bulk_wait<0>();
    } else {
        // ---- consumers -----------------------------------------------------------------------------------
        const int rl = tid >> 4, cg = tid & 15;             // K/V tiles: row lane and 16-byte column group
        float kacc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        TileIt it(a, b, cta, cps, nItems);
        Tile t;
        int slot = 0, j = 0;
        uint32_t phase = 0;
        bool ok = wait_on(&s_tab_ready, 0);
        while (it.next(&t)) {
            const unsigned char* sbase = ring + (size_t)slot * a.slotB;
            const int* td = s_tab_d[j & (kTabTiles - 1)];
            const float* tw = s_tab_w[j & (kTabTiles - 1)];
            if (ok) ok = wait_on(&s_full[slot], phase);
            if (ok && t.kv) {
                for (int p = rl; p < t.cnt; p += 16) {
                    if (td[p] != -1) continue;
                    const float wj = tw[p];
                    const uint4 xv = *reinterpret_cast<const uint4*>(sbase + p * kKvRowBytes + cg * 16);
                    kacc[0] = fmaf(wj, bf16_lo(xv.x), kacc[0]); kacc[1] = fmaf(wj, bf16_hi(xv.x), kacc[1]);
                    kacc[2] = fmaf(wj, bf16_lo(xv.y), kacc[2]); kacc[3] = fmaf(wj, bf16_hi(xv.y), kacc[3]);
                    kacc[4] = fmaf(wj, bf16_lo(xv.z), kacc[4]); kacc[5] = fmaf(wj, bf16_hi(xv.z), kacc[5]);
                    kacc[6] = fmaf(wj, bf16_lo(xv.w), kacc[6]); kacc[7] = fmaf(wj, bf16_hi(xv.w), kacc[7]);
                }
            } else if (ok && w) {
                for (int l = 0; l < t.cnt; ++l) {
                    if (td[l] != -1) continue;
                    const float wj = tw[l];
                    const uint4* rowp = reinterpret_cast<const uint4*>(sbase + (size_t)l * a.rowB);
#pragma unroll
                    for (int ci = 0; ci < CH; ++ci) {
                        const int c = tid + ci * kHidThreads;
                        if (c < a.V) {
                            const uint4 xv = rowp[c];
                            acc[ci][0] = fmaf(wj, bf16_lo(xv.x), acc[ci][0]); acc[ci][1] = fmaf(wj, bf16_hi(xv.x), acc[ci][1]);
                            acc[ci][2] = fmaf(wj, bf16_lo(xv.y), acc[ci][2]); acc[ci][3] = fmaf(wj, bf16_hi(xv.y), acc[ci][3]);
                            acc[ci][4] = fmaf(wj, bf16_lo(xv.z), acc[ci][4]); acc[ci][5] = fmaf(wj, bf16_hi(xv.z), acc[ci][5]);
                            acc[ci][6] = fmaf(wj, bf16_lo(xv.w), acc[ci][6]); acc[ci][7] = fmaf(wj, bf16_hi(xv.w), acc[ci][7]);
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) sm100::mbar_arrive(&s_empty[slot]);
            if (t.kv && t.item_end) {
                // end of a chunk: row lanes added in lane order, one partial row parked for the compaction kernel
#pragma unroll
                for (int e = 0; e < 8; ++e) { s_red[(rl * 16 + cg) * 8 + e] = kacc[e]; kacc[e] = 0.f; }
                asm volatile("bar.sync 1, %0;" ::"n"(kHidThreads) : "memory");
                if (tid < kHeadDim) {
                    float r = 0.f;
#pragma unroll
                    for (int l = 0; l < 16; ++l) r += s_red[l * kHeadDim + tid];
                    a.kv_partial[((int64_t)b * nItems + t.item) * kHeadDim + tid] = r;
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kHidThreads) : "memory");
            }
            ++j;
            if (++slot == S) { slot = 0; phase ^= 1u; }
        }
    }
    __syncthreads();
    if (s_abort) {                                             // copies may still be in flight: let them land
#pragma unroll 1
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (!w) return;                                            // no merged row in this mode

    // ---- the merged row of the hidden states --------------------------------------------------------------
    float* s_sum = reinterpret_cast<float*>(ring);            // [V][8] this CTA's sums; the ring is free now
    const int V = a.V, cl = a.cl;
    const int cluster = cta / cl;
    const int nq = cps / cl;                                   // partials of this sequence, one per cluster
    const int rank = (int)hid_cluster_rank();
    if (tid < kHidThreads) {
#pragma unroll
        for (int ci = 0; ci < CH; ++ci) {
            const int c = tid + ci * kHidThreads;
            if (c < V) {
                *reinterpret_cast<float4*>(s_sum + c * 8) = make_float4(acc[ci][0], acc[ci][1], acc[ci][2], acc[ci][3]);
                *reinterpret_cast<float4*>(s_sum + c * 8 + 4) = make_float4(acc[ci][4], acc[ci][5], acc[ci][6], acc[ci][7]);
            }
        }
    }
    hid_cluster_barrier();
    const int Vs = (V + cl - 1) / cl;                         // my slice of the column groups
    const int c_lo = min(V, rank * Vs), c_hi = min(V, c_lo + Vs);
    {
        // every CTA adds its slice of the columns over the CTAs of the cluster, in rank order
        float* my_partial = a.partial + ((int64_t)b * nq + cluster) * V * 8;
        for (int idx = tid; idx < (c_hi - c_lo) * 2; idx += kStreamThreads) {
            const int c = c_lo + (idx >> 1), half = idx & 1;
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int r = 0; r < cl; ++r) {
                const float4 x = hid_ld_cluster_f4(s_sum + c * 8 + half * 4, r);
                t.x += x.x; t.y += x.y; t.z += x.z; t.w += x.w;
            }
            *reinterpret_cast<float4*>(my_partial + c * 8 + half * 4) = t;
        }
    }
    hid_cluster_barrier();                 // every CTA's sums have been read: nobody leaves before
}

// Dynamic shared memory of the streaming kernel: always the whole ring budget, so that how many clusters fit on
// the GPU depends on the cluster size alone.
constexpr size_t kStreamSmem = (size_t)kStreamRingBytes;

template <int CH>
static lvlm_status launch_row_stream(const StreamArgs& a, int cps, int cl, int B, cudaStream_t stream) {
    LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(row_stream_kernel<CH>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem));
    return launch_kernel(row_stream_kernel<CH>, dim3((unsigned)cps, (unsigned)B), dim3(kStreamThreads), kStreamSmem,
                         stream, cl, a);
}

// How many clusters of `cl` CTAs of the streaming kernel the current device runs at a time (clusters are placed
// inside one GPC, so fewer CTAs fit than there are SMs); looked up once per device and cluster size.
template <int CH>
static int stream_clusters_resident(int cl) {
    static std::mutex mu;
    static int cache[64][4];                                // [device][log2 cl], 0 = not looked up yet
    int dev = 0, lg = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    while ((1 << lg) < cl) ++lg;
    std::lock_guard<std::mutex> lock(mu);
    if (cache[dev][lg] == 0) {
        if (cudaFuncSetAttribute(row_stream_kernel<CH>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem) !=
            cudaSuccess)
            return 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(cl * 64));
        cfg.blockDim = dim3(kStreamThreads);
        cfg.dynamicSmemBytes = kStreamSmem;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)cl; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, row_stream_kernel<CH>, &cfg) != cudaSuccess || n <= 0) {
            cudaGetLastError();
            n = 128 / cl;                                   // a safe guess
        }
        cache[dev][lg] = n;
    }
    return cache[dev][lg];
}

lvlm_status launch_hidden_rows(const void* hidden, void* hidden_out, int64_t hid_sb, int64_t out_sb,
                               const lvlm_dims* d, const HiddenGrid& L, const int32_t* dst_map,
                               const float* wgt, int32_t* meta, float* partial, void* scratch,
                               int64_t scr_sb, cudaStream_t stream, const StreamKv* kv, int32_t* dev_status,
                               int* partials_out) {
    const int chunks = (L.V + kHidThreads - 1) / kHidThreads;
    if (chunks > kHidMaxChunks || L.nstage < 3) return LVLM_ERR_UNSUPPORTED;  // more than 8192 channels
    // No more clusters than the device runs at a time: a second wave would double the time.  Clusters are placed
    // inside one GPC, so large clusters leave SMs idle: the cluster size is halved while that puts more CTAs to work
    // and the partial rows of a sequence stay few.
    int cps = 0, cl_run = L.cl;
    for (int cl = L.cl; cl >= 1; cl >>= 1) {
        int resident = 0;
        switch (chunks) {
            case 1: resident = stream_clusters_resident<1>(cl); break;
            case 2: resident = stream_clusters_resident<2>(cl); break;
            case 3: resident = stream_clusters_resident<3>(cl); break;
            case 4: resident = stream_clusters_resident<4>(cl); break;
        }
        int c = L.cps / cl * cl;
        if (resident > 0) {
            int per_seq = resident / d->B;
            per_seq = per_seq < 1 ? 1 : per_seq;
            if (c > per_seq * cl) c = per_seq * cl;
        }
        // (not for short sequences: there the extra partial rows cost more than the idle SMs)
        if (cl < L.cl && (c / cl > kMaxHidPartials || d->N < 48 * L.cps)) break;
        if (c > cps) { cps = c; cl_run = cl; }
    }
    if (partials_out) *partials_out = cps / cl_run;
    StreamArgs a;
    a.hid = static_cast<const char*>(hidden);
    a.out = static_cast<char*>(hidden_out);
    a.scratch = static_cast<char*>(scratch);
    a.hid_sb = hid_sb * 2; a.out_sb = out_sb * 2; a.scr_sb = scr_sb * 2;
    a.rowB = d->C * 2; a.V = L.V; a.N = d->N; a.i0 = d->i0; a.n = d->n; a.k = d->k; a.cl = cl_run;
    a.rpt = L.rpt; a.slotB = L.slotB; a.nstage = L.nstage;
    a.dst_map = dst_map; a.wgt = wgt; a.meta = meta; a.partial = partial;
    a.K = nullptr; a.Vc = nullptr; a.kv_sb = a.kv_sh = 0; a.Hkv = 0; a.kvP = 1; a.kvL = 1; a.kvT = 16;
    a.kv_partial = nullptr;
    if (kv && kv->K && wgt) {
        a.K = static_cast<const char*>(kv->K); a.Vc = static_cast<const char*>(kv->V);
        a.kv_sb = kv->kv_sb * 2; a.kv_sh = kv->kv_sh * 2; a.Hkv = kv->Hkv; a.kvP = kv->kvP;
        a.kvL = (d->n + kv->kvP - 1) / kv->kvP;
        a.kvT = L.slotB / kKvRowBytes >= 64 ? 64 : (L.slotB / kKvRowBytes) / 16 * 16;
        a.kv_partial = kv->kv_partial;
    }
    a.dev_status = dev_status;
    switch (chunks) {
        case 1: return launch_row_stream<1>(a, cps, cl_run, d->B, stream);
        case 2: return launch_row_stream<2>(a, cps, cl_run, d->B, stream);
        case 3: return launch_row_stream<3>(a, cps, cl_run, d->B, stream);
        case 4: return launch_row_stream<4>(a, cps, cl_run, d->B, stream);
    }
    return LVLM_ERR_UNSUPPORTED;
}

}  // namespace lvlm

extern "C" lvlm_status lvlm_merge_compact(void* hidden, void* hidden_out, void* Kc, void* Vc,
                                           int32_t* pos_ids, const int32_t* rank,
                                           const lvlm_dims* d, lvlm_merge_mode mode,
                                           const float* w_custom, float* mass, int32_t* new_len,
                                           void* ws, size_t ws_bytes, int32_t* dev_status,
                                           void* stream_) {
    using namespace lvlm;
    (void)mass;
    cudaStream_t stream = (cudaStream_t)stream_;
    MergeLayout L;
    if (!hidden || !rank || !merge_layout(d, &L)) return LVLM_ERR_INVALID_ARG;
    if ((Kc == nullptr) != (Vc == nullptr)) return LVLM_ERR_INVALID_ARG;
    if ((int)mode < 0 || (int)mode > LVLM_W_NEAREST_KEPT) return LVLM_ERR_INVALID_ARG;
    if (mode == LVLM_W_CUSTOM && !w_custom) return LVLM_ERR_INVALID_ARG;
    if (Kc) {
        if (d->Hkv <= 0 || d->cap < d->N) return LVLM_ERR_INVALID_ARG;
        if (d->D != kHeadDim) return LVLM_ERR_UNSUPPORTED;
    }
    if (mode == LVLM_W_NEAREST_KEPT) {    // no P_new row: N - (n - k) rows come out
        L.r = d->n - d->k;
        L.Nout = d->N - L.r;
    }
    const int64_t hid_sb = d->hid_stride_b ? d->hid_stride_b : (int64_t)d->N * d->C;
    if (hidden_out == hidden && mode != LVLM_W_NEAREST_KEPT) hidden_out = nullptr;   // the same buffer: compact in place
    const int64_t out_sb = hidden_out ? (d->out_stride_b ? d->out_stride_b : (int64_t)L.Nout * d->C) : hid_sb;
    const int64_t kv_sh = d->kv_stride_h ? d->kv_stride_h : (int64_t)d->cap * d->D;
    const int64_t kv_sb = d->kv_stride_b ? d->kv_stride_b : (int64_t)d->Hkv * kv_sh;
    if (!aligned16(hidden) || !aligned16(hidden_out) || !aligned16(Kc) || !aligned16(Vc) ||
        hid_sb % 8 || out_sb % 8 || kv_sh % 8 || kv_sb % 8)
        return LVLM_ERR_ALIGNMENT;
    if (hid_sb < (int64_t)d->N * d->C || out_sb < (int64_t)L.Nout * d->C) return LVLM_ERR_INVALID_ARG;
    if (hidden_out) {     // a separate output must not overlap the input: rows are read and written in no fixed order
        const char* in0 = static_cast<const char*>(hidden);
        const char* in1 = in0 + ((int64_t)(d->B - 1) * hid_sb + (int64_t)d->N * d->C) * 2;
        const char* out0 = static_cast<const char*>(hidden_out);
        const char* out1 = out0 + ((int64_t)(d->B - 1) * out_sb + (int64_t)L.Nout * d->C) * 2;
        if (out0 < in1 && in0 < out1) return LVLM_ERR_INVALID_ARG;
    }

    if (L.r <= 0) {                       // keep 100 %: every tensor stays as it is
        if (hidden_out && hidden_out != hidden) {
            LVLM_RETURN_IF_CUDA(cudaMemcpy2DAsync(hidden_out, out_sb * 2, hidden, hid_sb * 2,
                                                  (size_t)d->N * d->C * 2, d->B,
                                                  cudaMemcpyDeviceToDevice, stream));
        }
        if (new_len) return launch_kernel(identity_len_kernel, dim3((d->B + 127) / 128), dim3(128), 0, stream, 1,
                                          new_len, d->B, d->N);
        return LVLM_OK;
    }
    if (mode == LVLM_W_NEAREST_KEPT)
        return launch_nearest_kept(hidden, hidden_out, Kc, Vc, pos_ids, rank, d, mass, new_len, ws, ws_bytes,
                                   dev_status, stream);
    if (!ws || !aligned256(ws) || ws_bytes < L.total) return LVLM_ERR_WORKSPACE;
    char* wsb = static_cast<char*>(ws);
    int32_t* src_map = reinterpret_cast<int32_t*>(wsb + L.off_src);
    int32_t* dst_map = reinterpret_cast<int32_t*>(wsb + L.off_dst);
    float* wgt = reinterpret_cast<float*>(wsb + L.off_wgt);
    int32_t* meta = reinterpret_cast<int32_t*>(wsb + L.off_meta);
    float* partial = reinterpret_cast<float*>(wsb + L.off_partial);

    float inv_sum = 1.f;
    if (mode == LVLM_W_LINEAR_RANK) inv_sum = (float)(2.0 / ((double)L.r1 * ((double)L.r1 + 1.0)));
    else if (mode == LVLM_W_UNIFORM) inv_sum = (float)(1.0 / (double)L.r1);
    const int plan_threads = d->n >= 1024 ? 1024 : (d->n <= 128 ? 128 : ((d->n + 31) / 32) * 32);
    {
        int P = (d->n + 2047) / 2048;                    // CTAs per sequence: about two tiles of tokens each
        P = P < 1 ? 1 : (P > 8 ? 8 : P);
        const lvlm_status st = launch_kernel(merge_plan_kernel, dim3(P, d->B), dim3(plan_threads), 0, stream, P,
                                             rank, pos_ids, d->N, d->i0, d->n, d->k, (int)mode, inv_sum, w_custom,
                                             src_map, dst_map, wgt, meta, new_len, dev_status);
        if (st != LVLM_OK) return st;
    }

    float* kv_partial = reinterpret_cast<float*>(wsb + L.off_kvpartial);
    StreamKv kv = {Kc, Vc, kv_sb, kv_sh, d->Hkv, L.kvP, kv_partial};
    int hid_partials = L.grid.cps / L.grid.cl;
    {
        // one pass over the rows: kept hidden rows to their place (out of place only), merged rows of the hidden
        // states and of K and V into fp32 sums
        const lvlm_status st = launch_hidden_rows(hidden, hidden_out, hid_sb, out_sb, d, L.grid, dst_map, wgt, meta,
                                                  partial, nullptr, 0, stream, Kc ? &kv : nullptr, dev_status,
                                                  &hid_partials);
        if (st != LVLM_OK) return st;
    }
    // P_new of the hidden states: the partial rows are added by the compaction launch that follows
    if (!hidden_out) {
        CompactJob j;
        j.base0 = hidden; j.stride_b = hid_sb * 2; j.B = d->B; j.G = 1; j.V = L.V;
        j.src_map = src_map; j.map_stride = d->N; j.meta = meta; j.meta_stride = kMetaInts;
        j.Nout = L.Nout; j.N = d->N; j.merged_row = d->i0 + d->k; j.partial = partial;
        j.P = hid_partials; j.maps_ready = true;
        const lvlm_status st = launch_inplace_compact(j, stream);
        if (st != LVLM_OK) return st;
    }
    CompactJob j;
    if (hidden_out) {
        j.fin_base = hidden_out; j.fin_stride_b = out_sb * 2; j.fin_row = d->i0 + d->k; j.fin_V = L.V;
        j.fin_partial = partial; j.fin_P = hid_partials;
    }
    if (Kc) {
        j.base0 = Kc; j.base1 = Vc; j.stride_b = kv_sb * 2; j.stride_g = kv_sh * 2; j.G = d->Hkv;
        j.V = kHeadDim / 8;
        j.src_map = src_map; j.map_stride = d->N; j.meta = meta; j.meta_stride = kMetaInts;
        j.Nout = L.Nout; j.merged_row = d->i0 + d->k; j.partial = kv_partial; j.P = L.kvP;
    }
    j.B = d->B; j.N = d->N; j.maps_ready = true;
    if (Kc || hidden_out) {
        const lvlm_status st = launch_inplace_compact(j, stream);
        if (st != LVLM_OK) return st;
    }
    return LVLM_OK;
}
