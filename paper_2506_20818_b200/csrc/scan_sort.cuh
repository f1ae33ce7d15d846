// Integer primitives: exclusive scan, stable LSD radix sort of (key, value) pairs and the
// stable CSR transpose built on them.  Everything is integer work, so every result is unique
// and reproducible bit for bit.
#pragma once
#include "common.cuh"

// Optional per-category timing with CUDA events on the launching stream (lp_profile_begin/_end).
struct Profiler {
    uint32_t mask = 0;  // categories being timed; 0 = off
    uint32_t period = 1;  // only every period-th training step is timed
    uint64_t tick = 0;    // training steps seen
    bool live(int cat) const { return (mask & (1u << cat)) && (period <= 1 || tick % period == 0); }
    struct Span { int cat; cudaEvent_t a, b; double bytes, flops; };
    std::vector<Span> spans;
    std::vector<cudaEvent_t> pool;
    size_t used = 0;
    cudaEvent_t get()
    {
        if (used == pool.size()) {
            cudaEvent_t e = nullptr;
            cudaEventCreate(&e);
            pool.push_back(e);
        }
        return pool[used++];
    }
};

struct OnePassScan;
struct Exec {
    cudaStream_t st = nullptr;
    int64_t launches = 0;
    Profiler prof;
    OnePassScan *scan1 = nullptr;  // scratch of the one-launch scan (null: every scan takes three launches)
    int *scan_err = nullptr;       // device word that receives bit 1 when a bounded wait of that scan expires
};

// Times everything enqueued on the stream between construction and destruction when the category
// is selected; `bytes` / `flops` are the algorithmic figures of the enclosed launches.
struct ProfScope {
    Exec &ex;
    int idx = -1;
    ProfScope(Exec &e, int cat, double bytes = 0.0, double flops = 0.0) : ex(e)
    {
        if (ex.prof.live(cat)) {
            Profiler::Span s{cat, ex.prof.get(), ex.prof.get(), bytes, flops};
            cudaEventRecord(s.a, ex.st);
            idx = (int)ex.prof.spans.size();
            ex.prof.spans.push_back(s);
        }
    }
    ~ProfScope()
    {
        if (idx >= 0) cudaEventRecord(ex.prof.spans[idx].b, ex.st);
    }
};

// ------------------------------------------------------------------------------------------
// exclusive scan of int32 (three launches: tile sums, scan of the sums, rescan with offsets)
// ------------------------------------------------------------------------------------------
constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = 8;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;

LP_DEVINL int block_exclusive_scan_256(int x, int *smem_warp /*>=8 ints*/, int *total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    if (lane == 31) smem_warp[warp] = incl;
    __syncthreads();
    int base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < SCAN_THREADS / 32; ++w) {
        int s = smem_warp[w];
        if (w < warp) base += s;
        tot += s;
    }
    __syncthreads();
    *total = tot;
    return base + incl - x;
}

__global__ void __launch_bounds__(SCAN_THREADS) scan_tile_sums_kernel(const int *__restrict__ in, int64_t n, int *__restrict__ sums)
{
    LP_DEP_ENTER();
    __shared__ int sw[8];
    const int64_t base = (int64_t)blockIdx.x * SCAN_TILE;
    int acc = 0;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        int64_t idx = base + (int64_t)i * SCAN_THREADS + threadIdx.x;
        if (idx < n) acc += in[idx];
    }
    int tot;
    block_exclusive_scan_256(acc, sw, &tot);
    if (threadIdx.x == 0) sums[blockIdx.x] = tot;
}

// one block scans `m` values in place (exclusive), writes the grand total to *total if non-null
__global__ void __launch_bounds__(SCAN_THREADS) scan_single_block_kernel(int *__restrict__ data, int64_t m, int *__restrict__ total)
{
    LP_DEP_ENTER();
    __shared__ int sw[8];
    __shared__ int carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    for (int64_t base = 0; base < m; base += SCAN_TILE) {
        int v[SCAN_ITEMS];
        int acc = 0;
        const int64_t t0 = base + (int64_t)threadIdx.x * SCAN_ITEMS;
#pragma unroll
        for (int i = 0; i < SCAN_ITEMS; ++i) {
            v[i] = (t0 + i < m) ? data[t0 + i] : 0;
            acc += v[i];
        }
        int tot;
        int ex = block_exclusive_scan_256(acc, sw, &tot) + carry_s;
#pragma unroll
        for (int i = 0; i < SCAN_ITEMS; ++i) {
            if (t0 + i < m) data[t0 + i] = ex;
            ex += v[i];
        }
        __syncthreads();
        if (threadIdx.x == 0) carry_s += tot;
        __syncthreads();
    }
    if (total && threadIdx.x == 0) *total = carry_s;
}

__global__ void __launch_bounds__(SCAN_THREADS) scan_apply_kernel(const int *__restrict__ in, int64_t n, const int *__restrict__ tile_off,
                                                                  int *__restrict__ out, int *__restrict__ out_total)
{
    LP_DEP_ENTER();
    __shared__ int sw[8];
    const int64_t t0 = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
    int v[SCAN_ITEMS];
    int acc = 0;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        v[i] = (t0 + i < n) ? in[t0 + i] : 0;
        acc += v[i];
    }
    int tot;
    int ex = block_exclusive_scan_256(acc, sw, &tot) + tile_off[blockIdx.x];
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        if (t0 + i < n) out[t0 + i] = ex;
        ex += v[i];
    }
    // out[n] = total (the array has n+1 slots when out_total points at out + n)
    if (out_total && blockIdx.x == gridDim.x - 1 && threadIdx.x == SCAN_THREADS - 1) *out_total = ex;
}

static bool scan_onepass_try(Exec &ex, const int *in, int64_t n, int *out, int *out_copy, int *out_total);

// out[i] = sum_{j<i} in[j] for i in [0, n); if out_total != nullptr it receives the sum of all.
// `tmp` needs ceil(n / SCAN_TILE) + 1 ints.  in == out is allowed.  One launch when the context has the scratch of the
// one-launch scan and the input fits it, else three.
static void exclusive_scan_i32(Exec &ex, const int *in, int64_t n, int *out, int *out_total, int *tmp)
{
    if (n > 0 && scan_onepass_try(ex, in, n, out, nullptr, out_total)) return;
    if (n <= 0) {
        if (out_total) cudaMemsetAsync(out_total, 0, sizeof(int), ex.st);
        return;
    }
    const int64_t tiles = ceil_div64(n, SCAN_TILE);
    launch_dep(scan_tile_sums_kernel, dim3((unsigned)tiles), dim3(SCAN_THREADS), 0, ex.st, in, n, tmp);
    launch_dep(scan_single_block_kernel, dim3(1), dim3(SCAN_THREADS), 0, ex.st, tmp, tiles, nullptr);
    launch_dep(scan_apply_kernel, dim3((unsigned)tiles), dim3(SCAN_THREADS), 0, ex.st, in, n, tmp, out, out_total);
    ex.launches += 3;
}

// ------------------------------------------------------------------------------------------
// The same scan in ONE launch (for the scans inside a training step, where three dependent launches cost more
// than the work).  Tiles are handed out by a ticket, so a block only ever waits for tiles whose blocks are
// already running; a tile publishes its own sum at once and its inclusive prefix as soon as the look-back over its
// predecessors (one warp, 32 predecessors at a time) has found one.  A tile's status word carries the call's epoch,
// so the array needs no clearing between calls.  Every wait is bounded: on expiry bit 1 of *err is set, the tile
// carries on with what it has (the result of that call is wrong, the host reports it) and nothing hangs.
// ------------------------------------------------------------------------------------------
struct OnePassScan {
    unsigned long long *status = nullptr;  // one word per tile: epoch << 34 | flag << 32 | value (flag 1 = tile sum, 2 = inclusive prefix)
    unsigned *ticket = nullptr;            // next tile; the block that takes the last tile puts it back to 0
    int64_t tiles_cap = 0;
    unsigned epoch = 0;                    // host side: incremented by every call
};

LP_DEVINL unsigned long long scan_status_load(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
LP_DEVINL void scan_status_store(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

__global__ void __launch_bounds__(SCAN_THREADS) scan_onepass_kernel(const int *__restrict__ in, int64_t n, int *__restrict__ out, int *__restrict__ out_copy,
                                                                    int *__restrict__ out_total, unsigned long long *__restrict__ status,
                                                                    unsigned *__restrict__ ticket, unsigned epoch, int *__restrict__ err)
{
    LP_DEP_ENTER();
    __shared__ int sw[8];
    __shared__ unsigned tile_s;
    __shared__ int prefix_s;
    if (threadIdx.x == 0) {
        tile_s = atomicAdd(ticket, 1u);
        if (tile_s == gridDim.x - 1) *ticket = 0;  // every tile of this launch has been handed out
    }
    __syncthreads();
    const unsigned tile = tile_s;
    const int64_t t0 = (int64_t)tile * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
    int v[SCAN_ITEMS];
    int acc = 0;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        v[i] = (t0 + i < n) ? in[t0 + i] : 0;
        acc += v[i];
    }
    int tot;
    int ex = block_exclusive_scan_256(acc, sw, &tot);
    const unsigned long long tag = (unsigned long long)epoch << 34;
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        if (lane == 0) scan_status_store(status + tile, tag | ((tile == 0 ? 2ull : 1ull) << 32) | (unsigned)tot);
        int exclusive = 0;
        int64_t base = (int64_t)tile - 1;
        bool done = tile == 0;
        while (!done) {
            const int64_t t = base - lane;
            int flag = 2, val = 0;  // before the first tile: an inclusive prefix of 0
            if (t >= 0) {
                unsigned long long w = scan_status_load(status + t);
                if ((w >> 34) != epoch || ((w >> 32) & 3ull) == 0) {
                    unsigned long long t_start;
                    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_start));
                    for (;;) {
                        w = scan_status_load(status + t);
                        if ((w >> 34) == epoch && ((w >> 32) & 3ull) != 0) break;
                        unsigned long long now;
                        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(now));
                        if (now - t_start > 2000000000ull) {  // two seconds: give up, report, carry on
                            atomicOr(err, 2);
                            w = tag | (2ull << 32);
                            break;
                        }
                    }
                }
                flag = (int)((w >> 32) & 3ull);
                val = (int)(unsigned)(w & 0xffffffffull);
            }
            const unsigned has_prefix = __ballot_sync(0xffffffffu, flag == 2);
            const int upto = has_prefix ? __ffs(has_prefix) - 1 : 31;  // nearest predecessor that knows its inclusive prefix
            int contrib = lane <= upto ? val : 0;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) contrib += __shfl_xor_sync(0xffffffffu, contrib, o);
            exclusive += contrib;
            if (has_prefix) done = true; else base -= 32;
        }
        if (lane == 0) {
            prefix_s = exclusive;
            if (tile != 0) scan_status_store(status + tile, tag | (2ull << 32) | (unsigned)(exclusive + tot));
        }
    }
    __syncthreads();
    ex += prefix_s;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        if (t0 + i < n) {
            out[t0 + i] = ex;
            if (out_copy) out_copy[t0 + i] = ex;
        }
        ex += v[i];
    }
    if (out_total && tile == gridDim.x - 1 && threadIdx.x == SCAN_THREADS - 1) *out_total = ex;
}

static bool scan_onepass_try(Exec &ex, const int *in, int64_t n, int *out, int *out_copy, int *out_total)
{
    OnePassScan *sc = ex.scan1;
    const int64_t tiles = ceil_div64(n, SCAN_TILE);
    if (!sc || !sc->status || tiles > sc->tiles_cap) return false;
    sc->epoch = (sc->epoch + 1u) & 0x3fffffffu;
    if (sc->epoch == 0) sc->epoch = 1;
    launch_dep(scan_onepass_kernel, dim3((unsigned)tiles), dim3(SCAN_THREADS), 0, ex.st, in, n, out, out_copy, out_total, sc->status, sc->ticket, sc->epoch, ex.scan_err);
    ex.launches += 1;
    return true;
}

// the same scan with a second copy of the result (out_copy), as the incidence lists want it (offsets and cursors)
static void exclusive_scan_i32_copy(Exec &ex, const int *in, int64_t n, int *out, int *out_copy, int *out_total, int *tmp)
{
    if (n <= 0) {
        if (out_total) cudaMemsetAsync(out_total, 0, sizeof(int), ex.st);
        return;
    }
    if (scan_onepass_try(ex, in, n, out, out_copy, out_total)) return;
    exclusive_scan_i32(ex, in, n, out, out_total, tmp);
    cudaMemcpyAsync(out_copy, out, sizeof(int) * (size_t)n, cudaMemcpyDeviceToDevice, ex.st);
}

// ------------------------------------------------------------------------------------------
// stable LSD radix sort of pairs, 8 bits per pass
// ------------------------------------------------------------------------------------------
constexpr int RS_THREADS = 256;
constexpr int RS_ROUNDS = 8;
constexpr int RS_TILE = RS_THREADS * RS_ROUNDS;
constexpr int RS_RADIX = 256;

__global__ void __launch_bounds__(RS_THREADS) rs_hist_kernel(const uint32_t *__restrict__ keys, int64_t n, int shift,
                                                             int *__restrict__ hist /*[RADIX][tiles]*/, int tiles)
{
    LP_DEP_ENTER();
    __shared__ int h[RS_RADIX];
    h[threadIdx.x] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * RS_TILE;
#pragma unroll
    for (int r = 0; r < RS_ROUNDS; ++r) {
        int64_t idx = base + r * RS_THREADS + threadIdx.x;
        if (idx < n) atomicAdd(&h[(keys[idx] >> shift) & (RS_RADIX - 1)], 1);
    }
    __syncthreads();
    hist[(int64_t)threadIdx.x * tiles + blockIdx.x] = h[threadIdx.x];
}

__global__ void __launch_bounds__(RS_THREADS) rs_scatter_kernel(const uint32_t *__restrict__ keys, const uint32_t *__restrict__ vals,
                                                                int64_t n, int shift, const int *__restrict__ hist_scanned, int tiles,
                                                                uint32_t *__restrict__ keys_out, uint32_t *__restrict__ vals_out)
{
    LP_DEP_ENTER();
    __shared__ int base[RS_RADIX];                    // next free output slot per digit for this tile
    __shared__ int wcount[RS_THREADS / 32][RS_RADIX]; // per-warp digit counts of the current round
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    base[threadIdx.x] = hist_scanned[(int64_t)threadIdx.x * tiles + blockIdx.x];
    const int64_t tbase = (int64_t)blockIdx.x * RS_TILE;
    for (int r = 0; r < RS_ROUNDS; ++r) {
#pragma unroll
        for (int w = 0; w < RS_THREADS / 32; ++w) wcount[w][threadIdx.x] = 0;
        __syncthreads();
        const int64_t idx = tbase + r * RS_THREADS + threadIdx.x;
        const bool valid = idx < n;
        uint32_t key = valid ? keys[idx] : 0xFFFFFFFFu;
        uint32_t val = valid ? vals[idx] : 0u;
        // invalid lanes take a digit of their own (RADIX) so they never match valid ones
        const int digit = valid ? (int)((key >> shift) & (RS_RADIX - 1)) : RS_RADIX;
        const unsigned peers = __match_any_sync(0xffffffffu, digit);
        const int rank_in_warp = __popc(peers & ((1u << lane) - 1u));
        if (valid && rank_in_warp == 0) wcount[warp][digit] = __popc(peers);
        __syncthreads();
        if (valid) {
            int pos = base[digit] + rank_in_warp;
            for (int w = 0; w < warp; ++w) pos += wcount[w][digit];
            keys_out[pos] = key;
            vals_out[pos] = val;
        }
        __syncthreads();
        {
            int add = 0;
#pragma unroll
            for (int w = 0; w < RS_THREADS / 32; ++w) add += wcount[w][threadIdx.x];
            base[threadIdx.x] += add;
        }
        __syncthreads();
    }
}

struct SortScratch {  // caller-provided device buffers
    uint32_t *keys_alt = nullptr, *vals_alt = nullptr;  // n entries each
    int *hist = nullptr;                                // RADIX * ceil(n / RS_TILE) + 1 ints
    int *scan_tmp = nullptr;                            // ceil(hist entries / SCAN_TILE) + 1 ints
    static int64_t hist_ints(int64_t n) { return (int64_t)RS_RADIX * ceil_div64(n > 0 ? n : 1, RS_TILE) + 1; }
    static int64_t scan_ints(int64_t n) { return ceil_div64(hist_ints(n), SCAN_TILE) + 1; }
};

// Sorts (keys, vals) by the low `key_bits` bits of the key, stably, in ceil(key_bits / 8) passes.
// Returns true when the result is in (keys, vals), false when it is in (s.keys_alt, s.vals_alt).
static bool radix_sort_pairs(Exec &ex, uint32_t *keys, uint32_t *vals, int64_t n, int key_bits, const SortScratch &s)
{
    if (n <= 0) return true;
    int passes = (key_bits + 7) / 8;
    if (passes < 1) passes = 1;
    const int tiles = (int)ceil_div64(n, RS_TILE);
    uint32_t *ki = keys, *vi = vals, *ko = s.keys_alt, *vo = s.vals_alt;
    for (int p = 0; p < passes; ++p) {
        launch_dep(rs_hist_kernel, dim3(tiles), dim3(RS_THREADS), 0, ex.st, ki, n, 8 * p, s.hist, tiles);
        ex.launches += 1;
        exclusive_scan_i32(ex, s.hist, (int64_t)RS_RADIX * tiles, s.hist, nullptr, s.scan_tmp);
        launch_dep(rs_scatter_kernel, dim3(tiles), dim3(RS_THREADS), 0, ex.st, ki, vi, n, 8 * p, s.hist, tiles, ko, vo);
        ex.launches += 1;
        uint32_t *t;
        t = ki; ki = ko; ko = t;
        t = vi; vi = vo; vo = t;
    }
    return ki == keys;
}

// ------------------------------------------------------------------------------------------
// CSR transpose pieces
// ------------------------------------------------------------------------------------------
// keys[e] = col[e], vals[e] = e, rows[e] = row of entry e (one thread per entry; row found by
// binary search over rowptr)
__global__ void expand_entries_kernel(const int *__restrict__ rowptr, int n_rows, const int *__restrict__ col, int64_t nnz,
                                      uint32_t *__restrict__ keys, uint32_t *__restrict__ vals, int *__restrict__ rows)
{
    LP_DEP_ENTER();
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= nnz) return;
    int lo = 0, hi = n_rows;  // largest r with rowptr[r] <= e
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if ((int64_t)rowptr[mid] <= e) lo = mid; else hi = mid;
    }
    keys[e] = (uint32_t)col[e];
    vals[e] = (uint32_t)e;
    rows[e] = lo;
}

// the same when the row of every entry is already known: keys, values and the per-column counts in one pass
__global__ void expand_known_rows_kernel(const int *__restrict__ col, int64_t nnz, uint32_t *__restrict__ keys, uint32_t *__restrict__ vals,
                                         int *__restrict__ counts)
{
    LP_DEP_ENTER();
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= nnz) return;
    const int c = col[e];
    keys[e] = (uint32_t)c;
    vals[e] = (uint32_t)e;
    atomicAdd(&counts[c], 1);
}

__global__ void count_keys_kernel(const int *__restrict__ ids, int64_t m, int *__restrict__ counts)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < m) atomicAdd(&counts[ids[i]], 1);
}

__global__ void gather_rows_kernel(const uint32_t *__restrict__ sorted_vals, const int *__restrict__ rows, int64_t nnz,
                                   int *__restrict__ rowidx_t, int *__restrict__ perm)
{
    LP_DEP_ENTER();
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= nnz) return;
    const uint32_t e = sorted_vals[t];
    rowidx_t[t] = rows[e];
    perm[t] = (int)e;
}

static int bits_for(int64_t n)
{
    int b = 1;
    while (((int64_t)1 << b) < n) ++b;
    return b;
}

struct TransposeScratch {
    uint32_t *keys = nullptr, *vals = nullptr;  // nnz each
    int *rows = nullptr;                        // nnz
    SortScratch sort;
    int *scan_tmp = nullptr;                    // ceil(n_cols / SCAN_TILE) + 1
};

// Stable transpose of a CSR with n_rows rows and n_cols columns: colptr[n_cols + 1],
// rowidx_t[nnz] (row of each transposed entry, ascending inside a transposed row because the
// sort is stable and entries are visited in row order) and perm[nnz] (original entry index).
static void transpose_csr(Exec &ex, const int *rowptr, int n_rows, int n_cols, const int *col, int64_t nnz, int *colptr,
                          int *rowidx_t, int *perm, const TransposeScratch &s, const int *rows_known = nullptr)
{
    cudaMemsetAsync(colptr, 0, sizeof(int) * ((size_t)n_cols + 1), ex.st);
    if (nnz > 0) {
        const unsigned blocks = (unsigned)ceil_div64(nnz, 256);
        if (rows_known) {  // the caller has the row of every entry (sampled blocks record it)
            launch_dep(expand_known_rows_kernel, dim3(blocks), dim3(256), 0, ex.st, col, nnz, s.keys, s.vals, colptr);
            ex.launches += 1;
        } else {
            launch_dep(expand_entries_kernel, dim3(blocks), dim3(256), 0, ex.st, rowptr, n_rows, col, nnz, s.keys, s.vals, s.rows);
            launch_dep(count_keys_kernel, dim3(blocks), dim3(256), 0, ex.st, col, nnz, colptr);
            ex.launches += 2;
        }
    }
    exclusive_scan_i32(ex, colptr, n_cols, colptr, colptr + n_cols, s.scan_tmp);
    if (nnz > 0) {
        const bool in_place = radix_sort_pairs(ex, s.keys, s.vals, nnz, bits_for(n_cols), s.sort);
        launch_dep(gather_rows_kernel, dim3((unsigned)ceil_div64(nnz, 256)), dim3(256), 0, ex.st, in_place ? s.vals : s.sort.vals_alt, rows_known ? rows_known : s.rows, nnz, rowidx_t, perm);
        ex.launches += 1;
    }
}
