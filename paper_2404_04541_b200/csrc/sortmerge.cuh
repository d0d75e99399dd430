// Sort and Merge stages shared by the workspaces that keep their accumulation array and all array
// in global memory (Algorithm 1 with integer labels, Sec. 5.2): a stable LSD radix sort of 64-bit
// labels with the values carried along, the reduction of runs of equal labels in insertion
// order, and the driver that feeds the products in rounds of the accumulation array's capacity.
// Included by the translation units that instantiate it.
#pragma once
#include "common.cuh"

namespace spws {

constexpr int OT = 256;                 // threads of the element-wise kernels
constexpr u64 ABSENT_LABEL = ~0ull;     // a numbered product that does not exist (sorts last, dropped)

static int grid_for(const LaunchCtx& c, i64 work_items, int per_block) {
    i64 want = (work_items + per_block - 1) / per_block;
    const i64 cap = (i64)c.sm_count * 16;
    if (want > cap) want = cap;
    return (int)(want < 1 ? 1 : want);
}

// ---- stable LSD radix sort, 8 bits per pass -------------------------------------------------
// A block owns a tile of RS_TILE consecutive elements; warp w of the block owns the w-th
// contiguous slice of the tile and walks it 32 elements at a time, so "block, warp, step, lane"
// is the input order.  Pass = histogram per (digit, block) -> exclusive scan over (digit major,
// block minor) -> scatter with the element's rank among equal digits before it; the tile is put in
// digit order in shared memory first, so every digit's elements leave as one contiguous run.
constexpr int RS_THREADS = 256;
constexpr int RS_WARPS = RS_THREADS / 32;
constexpr int RS_STEPS = 8;                             // 32-element steps per warp
constexpr int RS_TILE = RS_WARPS * RS_STEPS * 32;       // 2048

static __global__ void __launch_bounds__(RS_THREADS) radix_hist_kernel(const u64* __restrict__ keys, i64 n, int shift, int nblocks,
                                                               int* __restrict__ hist) {
    __shared__ int s_h[256];
    s_h[threadIdx.x] = 0;
    __syncthreads();
    const i64 base = (i64)blockIdx.x * RS_TILE;
    for (int x = threadIdx.x; x < RS_TILE; x += RS_THREADS)
        if (base + x < n) atomicAdd(&s_h[(keys[base + x] >> shift) & 255], 1);
    __syncthreads();
    hist[(i64)threadIdx.x * nblocks + blockIdx.x] = s_h[threadIdx.x];
}

template <typename T, bool VALUES>
__global__ void __launch_bounds__(RS_THREADS) radix_scatter_kernel(const u64* __restrict__ keys, const T* __restrict__ vals, i64 n,
                                                                  int shift, int nblocks, const i64* __restrict__ offs,
                                                                  u64* __restrict__ keys_out, T* __restrict__ vals_out) {
    __shared__ int s_cnt[RS_WARPS][256];        // elements with the digit in this warp's slice, then their start inside the digit's part
    __shared__ int s_start[256];                // start of the digit's part inside the tile
    __shared__ i64 s_goff[256];
    __shared__ int s_ws[33];
    __shared__ u64 s_key[RS_TILE];
    __shared__ T s_val[VALUES ? RS_TILE : 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int d = lane; d < 256; d += 32) s_cnt[warp][d] = 0;
    __syncwarp();
    const i64 base = (i64)blockIdx.x * RS_TILE + (i64)warp * (RS_STEPS * 32);
    u64 key[RS_STEPS];
    int rank[RS_STEPS];
#pragma unroll
    for (int st = 0; st < RS_STEPS; ++st) {
        const i64 t = base + st * 32 + lane;
        const bool live = t < n;
        key[st] = live ? keys[t] : ~0ull;
        const unsigned d = (unsigned)(key[st] >> shift) & 255u;
        // lanes of this step with the same digit (lanes past the end form their own group)
        const unsigned peers = __match_any_sync(0xffffffffu, live ? d : 256u);
        const int before = __popc(peers & ((1u << lane) - 1u));
        int old = 0;
        if (live && before == 0) {                       // first lane of a group books the group's slots
            old = s_cnt[warp][d];
            s_cnt[warp][d] = old + __popc(peers);
        }
        old = __shfl_sync(0xffffffffu, old, __ffs(peers) - 1);
        rank[st] = old + before;
        __syncwarp();
    }
    __syncthreads();
    // start of each warp's share of a digit inside the digit's part of the tile, and the start of
    // every digit's part inside the tile (the tile is first put in digit order in shared memory,
    // so that each digit's elements leave as one contiguous run)
    int tile_total;
    {
        const int d = threadIdx.x;                       // RS_THREADS == 256 digits
        int run = 0;
        for (int w = 0; w < RS_WARPS; ++w) { const int c = s_cnt[w][d]; s_cnt[w][d] = run; run += c; }
        const int start = block_excl_scan<RS_THREADS>(run, s_ws, tile_total);
        s_start[d] = start;
        s_goff[d] = offs[(i64)d * nblocks + blockIdx.x] - start;     // global position of staged slot i of digit d = s_goff[d] + i
    }
    __syncthreads();
#pragma unroll
    for (int st = 0; st < RS_STEPS; ++st) {
        const i64 t = base + st * 32 + lane;
        if (t < n) {
            const unsigned d = (unsigned)(key[st] >> shift) & 255u;
            const int at = s_start[d] + s_cnt[warp][d] + rank[st];
            s_key[at] = key[st];
            if (VALUES) s_val[at] = vals[t];
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < tile_total; i += RS_THREADS) {
        const u64 k = s_key[i];
        const i64 at = s_goff[(unsigned)(k >> shift) & 255u] + i;
        keys_out[at] = k;
        if (VALUES) vals_out[at] = s_val[i];
    }
}

// ---- Merge (reduce runs of equal labels) and Compress ----------------------------------------
static __global__ void __launch_bounds__(OT) heads_kernel(const u64* __restrict__ keys, i64 n, int* __restrict__ head) {
    for (i64 t = (i64)blockIdx.x * OT + threadIdx.x; t < n; t += (i64)gridDim.x * OT)
        head[t] = (t == 0 || keys[t] != keys[t - 1]) ? 1 : 0;
}

// Writes the duplicate-free sequence: label and (VALUES) the run's sum in insertion order.
template <typename T, bool VALUES>
__global__ void __launch_bounds__(OT) reduce_runs_kernel(const u64* __restrict__ keys, const T* __restrict__ vals, i64 n,
                                                         const int* __restrict__ head, const i64* __restrict__ at,
                                                         u64* __restrict__ ukeys, T* __restrict__ uvals) {
    for (i64 t = (i64)blockIdx.x * OT + threadIdx.x; t < n; t += (i64)gridDim.x * OT) {
        if (!head[t]) continue;
        const u64 key = keys[t];
        ukeys[at[t]] = key;
        if (VALUES) {
            T sum = vals[t];
            for (i64 y = t + 1; y < n && keys[y] == key; ++y) sum = add_rn(sum, vals[y]);
            uvals[at[t]] = sum;
        }
    }
}

// Sorts n (label, value) pairs by label; `bits` = number of significant label bits.  Input in
// (k0, v0), the other buffer in (k1, v1); *in_first tells which pair holds the result.
template <typename T, bool VALUES>
static cudaError_t radix_sort_t(const LaunchCtx& c, i64 n, int bits, u64* k0, T* v0, u64* k1, T* v1, char* tmp, bool* in_first) {
    *in_first = true;
    if (n <= 1) return cudaSuccess;
    const int nblocks = (int)((n + RS_TILE - 1) / RS_TILE);
    const size_t cells = (size_t)256 * (size_t)nblocks;
    int* hist = reinterpret_cast<int*>(tmp);
    i64* offs = reinterpret_cast<i64*>(tmp + ((cells * 4 + 255) & ~(size_t)255));
    i64* block_sums = reinterpret_cast<i64*>(reinterpret_cast<char*>(offs) + (((cells + 1) * 8 + 255) & ~(size_t)255));
    u64 *ki = k0, *ko = k1;
    T *vi = v0, *vo = v1;
    for (int shift = 0; shift < bits; shift += 8) {
        radix_hist_kernel<<<nblocks, RS_THREADS, 0, c.stream>>>(ki, n, shift, nblocks, hist);
        ++c.launches;
        cudaError_t e = launch_scan_counts(c, hist, (int)cells, offs, block_sums, nullptr);
        if (e != cudaSuccess) return e;
        radix_scatter_kernel<T, VALUES><<<nblocks, RS_THREADS, 0, c.stream>>>(ki, vi, n, shift, nblocks, offs, ko, vo);
        ++c.launches;
        u64* tk = ki; ki = ko; ko = tk;
        T* tv = vi; vi = vo; vo = tv;
        *in_first = !*in_first;
    }
    return cudaGetLastError();
}

static __global__ void drop_absent_kernel(const u64* __restrict__ ukeys, i64* cnt) {
    if (*cnt > 0 && ukeys[*cnt - 1] == ABSENT_LABEL) --*cnt;
}

// Sort + reduce n entries that start at (k, v); the other buffer of the same size is (k2, v2).
// The duplicate-free result is written to (dst_k, dst_v), which must be one of the two buffers
// and not the one the sorted sequence ended in -- the caller passes both candidates and learns
// which was used.  The number of distinct labels goes to *cnt_dev and is read back.
template <typename T, bool VALUES>
static cudaError_t sort_reduce_t(const LaunchCtx& c, i64 n, int label_bits, u64* k, T* v, u64* k2, T* v2, int* head, i64* at,
                                 char* sort_tmp, i64* block_sums, i64* cnt_dev, i64* cnt_host_pinned, bool* result_in_first) {
    bool first = true;
    cudaError_t e = radix_sort_t<T, VALUES>(c, n, label_bits, k, v, k2, v2, sort_tmp, &first);
    if (e != cudaSuccess) return e;
    u64* ks = first ? k : k2;
    T* vs = first ? v : v2;
    u64* ku = first ? k2 : k;
    T* vu = first ? v2 : v;
    if (n > 0) {
        heads_kernel<<<grid_for(c, n, OT), OT, 0, c.stream>>>(ks, n, head);
        ++c.launches;
    }
    if ((e = launch_scan_counts(c, head, (int)n, at, block_sums, cnt_dev)) != cudaSuccess) return e;
    if (n > 0) {
        reduce_runs_kernel<T, VALUES><<<grid_for(c, n, OT), OT, 0, c.stream>>>(ks, vs, n, head, at, ku, vu);
        ++c.launches;
    }
    if (n > 0) {                        // absent products carry the largest label: one trailing entry at most
        drop_absent_kernel<<<1, 1, 0, c.stream>>>(ku, cnt_dev);
        ++c.launches;
    }
    if ((e = cudaMemcpyAsync(cnt_host_pinned, cnt_dev, sizeof(i64), cudaMemcpyDeviceToHost, c.stream)) != cudaSuccess) return e;
    if ((e = cudaStreamSynchronize(c.stream)) != cudaSuccess) return e;
    *result_in_first = !first;
    return cudaGetLastError();
}

// One pass of a sparse workspace over P numbered products, in rounds of `cap` (Algorithm 1: when
// the accumulation array is full it is sorted and reduced on its own, then united with the all
// array; the entry that found it full opens the next round).  `expand(t0, n, keys, vals)` enqueues
// the kernel that appends the products with ordinals [t0, t0 + n); a product may be marked absent
// with the all-ones label, which sorts last and is dropped.
// Buffers: two (label, value) arrays of N = P + (cap < P ? cap : 0) entries, head flags and
// their scan (N, N + 1), sort temporaries.  On return *result_first tells which array holds the
// duplicate-free result; its length is in *nnz_host_pinned.
template <typename T, bool VALUES, typename Expand>
static cudaError_t ism_rounds_t(const LaunchCtx& c, Expand expand, i64 P, i64 cap, int label_bits,
                                u64* kA, T* vA, u64* kB, T* vB, int* head, i64* at, char* sort_tmp, i64* block_sums,
                                i64* nnz_dev, i64* nnz_host_pinned, bool* result_first) {
    u64 *kc = kA, *ko = kB;             // kc/vc: the buffer that holds the all array (n_all entries, sorted, duplicate-free)
    T *vc = vA, *vo = vB;
    i64 n_all = 0;
    *nnz_host_pinned = 0;
    const size_t vsz = VALUES ? sizeof(T) : 0;
    for (i64 t0 = 0; t0 < P; t0 += cap) {
        const i64 n_new = (P - t0 < cap) ? P - t0 : cap;
        // Insert: the round's products behind the all array
        cudaError_t e = expand(t0, n_new, kc + n_all, VALUES ? vc + n_all : (T*)nullptr);
        if (e != cudaSuccess) return e;
        // Sort + reduce of the accumulation array alone
        bool in_first = true;
        e = sort_reduce_t<T, VALUES>(c, n_new, label_bits, kc + n_all, VALUES ? vc + n_all : nullptr, ko + n_all,
                                     VALUES ? vo + n_all : nullptr, head, at, sort_tmp, block_sums, nnz_dev, nnz_host_pinned, &in_first);
        if (e != cudaSuccess) return e;
        const i64 n_acc = *nnz_host_pinned;
        if (n_all == 0) {
            // nothing to unite with: the reduced accumulation array is the all array
            if (!in_first) { u64* tk = kc; kc = ko; ko = tk; T* tv = vc; vc = vo; vo = tv; }
            n_all = n_acc;
            continue;
        }
        if (!in_first) {                // bring the reduced accumulation array behind the all array
            if ((e = cudaMemcpyAsync(kc + n_all, ko + n_all, 8 * (size_t)n_acc, cudaMemcpyDeviceToDevice, c.stream)) != cudaSuccess) return e;
            if (VALUES && (e = cudaMemcpyAsync(vc + n_all, vo + n_all, vsz * (size_t)n_acc, cudaMemcpyDeviceToDevice, c.stream)) != cudaSuccess) return e;
        }
        // Merge: all array first, so that a label in both sums as all + accumulated
        e = sort_reduce_t<T, VALUES>(c, n_all + n_acc, label_bits, kc, vc, ko, vo, head, at, sort_tmp, block_sums, nnz_dev, nnz_host_pinned, &in_first);
        if (e != cudaSuccess) return e;
        if (!in_first) { u64* tk = kc; kc = ko; ko = tk; T* tv = vc; vc = vo; vo = tv; }
        n_all = *nnz_host_pinned;
    }
    *nnz_host_pinned = n_all;
    *result_first = (kc == kA);
    return cudaGetLastError();
}

}  // namespace spws
