// Outer-product SpGEMM  C(i,j) = sum_k A(k,i) * B(k,j)  through a SECOND-ORDER workspace
// (Sec. 2.1 running example, Sec. 2.2: loop order k -> i -> j against output order i -> j makes
// both output coordinates scatter, so one workspace holds components of the whole result).
//
// Sparse workspace (Algorithm 1, coordinate-sort policy with integer labels, Sec. 5.2):
//   Insert   : the products are numbered in loop order (k, then the entries of A's row k, then
//              the entries of B's row k); a round takes the next `cap` of them and appends
//              (label = i * J + j, value) to the accumulation array in global memory.
//   Sort     : stable LSD radix sort of the labels, 8 bits per pass, values carried along.
//   Merge    : equal labels are adjacent and in insertion order: each run is summed in that order.
//              With several rounds the reduced accumulation array is united with the sorted,
//              duplicate-free all array by sorting the two together, all array first, so a label
//              present in both becomes all + accumulated.
//   Compress : row i's entries are the labels in [i*J, (i+1)*J): pos by binary search, crd = label
//              mod J.
// Dense workspace (Table 2's dense array + flags, second order): an I x J value array and an
// I x J-bit occupancy bitmap in global memory; products are added / flagged in place, rows are
// then counted, scanned and copied out in column order.
//
// A is given by its rows k (the CSR arrays of the K x I matrix whose (k,i) entry is A(k,i)).
#include "common.cuh"

namespace spws {

constexpr int OT = 256;                 // threads of the element-wise kernels

// ---- product numbering --------------------------------------------------------------------
__global__ void __launch_bounds__(OT) outer_counts_kernel(Csr At, Csr B, int* __restrict__ cnt, DevCtl* ctl) {
    for (i64 k = (i64)blockIdx.x * OT + threadIdx.x; k < At.nrows; k += (i64)gridDim.x * OT) {
        const i64 c = (At.pos[k + 1] - At.pos[k]) * (B.pos[k + 1] - B.pos[k]);
        if (c > 0x7fffffffll) { raise_status(ctl, DEV_INTERNAL_OVERFLOW); cnt[k] = 0; }
        else cnt[k] = (int)c;
    }
}

// The product with ordinal t belongs to the last k whose first ordinal is <= t.
__device__ __forceinline__ int owner_k(const i64* __restrict__ koff, int K, i64 t) {
    int lo = 0, hi = K;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (koff[mid] <= t) lo = mid; else hi = mid;
    }
    return lo;
}

// Appends the products with ordinals [t0, t0 + n) at out[dst0 ...): four consecutive ordinals per thread.
template <typename T, bool VALUES, bool DENSE>
__global__ void __launch_bounds__(OT) outer_expand_kernel(Csr At, Csr B, const i64* __restrict__ koff, i64 t0, i64 n, i64 J,
                                                          u64* __restrict__ keys, T* __restrict__ vals,
                                                          unsigned* __restrict__ dbits, T* __restrict__ dvals, i64 row_words,
                                                          DevCtl* ctl) {
    const T* __restrict__ Aval = (const T*)At.val;
    const T* __restrict__ Bval = (const T*)B.val;
    for (i64 s = ((i64)blockIdx.x * OT + threadIdx.x) * 4; s < n; s += (i64)gridDim.x * OT * 4) {
        i64 t = t0 + s;
        int k = owner_k(koff, At.nrows, t);
        for (int x = 0; x < 4 && s + x < n; ++x, ++t) {
            while (koff[k + 1] <= t) ++k;
            const i64 r = t - koff[k];
            const i64 lb = B.pos[k + 1] - B.pos[k];
            const i64 p = At.pos[k] + r / lb, q = B.pos[k] + r % lb;
            const int i = At.crd[p], j = B.crd[q];
            if ((unsigned)i >= (unsigned)At.ncols || (i64)j >= J || j < 0) { raise_status(ctl, DEV_NONCANONICAL); continue; }
            if (DENSE) {
                atomicOr(&dbits[(i64)i * row_words + (j >> 5)], 1u << (j & 31));
                if (VALUES) atomicAdd(&dvals[(i64)i * J + j], mul_rn(Aval[p], Bval[q]));
            } else {
                keys[s + x] = (u64)i * (u64)J + (u64)j;
                if (VALUES) vals[s + x] = mul_rn(Aval[p], Bval[q]);
            }
        }
    }
}

// ---- stable LSD radix sort, 8 bits per pass -------------------------------------------------
// A block owns a tile of RS_TILE consecutive elements; warp w of the block owns the w-th
// contiguous slice of the tile and walks it 32 elements at a time, so "block, warp, step, lane"
// is the input order.  Pass = histogram per (digit, block) -> exclusive scan over (digit major,
// block minor) -> scatter with the element's rank among equal digits before it.
constexpr int RS_THREADS = 256;
constexpr int RS_WARPS = RS_THREADS / 32;
constexpr int RS_STEPS = 8;                             // 32-element steps per warp
constexpr int RS_TILE = RS_WARPS * RS_STEPS * 32;       // 2048

__global__ void __launch_bounds__(RS_THREADS) radix_hist_kernel(const u64* __restrict__ keys, i64 n, int shift, int nblocks,
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
    __shared__ int s_cnt[RS_WARPS][256];        // elements with the digit in this warp's slice, then their start inside the tile
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
    // start of each warp's share of a digit = global start of (digit, block) + earlier warps' counts
    {
        const int d = threadIdx.x;                       // RS_THREADS == 256 digits
        int run = 0;
        for (int w = 0; w < RS_WARPS; ++w) { const int c = s_cnt[w][d]; s_cnt[w][d] = run; run += c; }
    }
    __syncthreads();
#pragma unroll
    for (int st = 0; st < RS_STEPS; ++st) {
        const i64 t = base + st * 32 + lane;
        if (t < n) {
            const unsigned d = (unsigned)(key[st] >> shift) & 255u;
            const i64 at = offs[(i64)d * nblocks + blockIdx.x] + s_cnt[warp][d] + rank[st];
            keys_out[at] = key[st];
            if (VALUES) vals_out[at] = vals[t];
        }
    }
}

// ---- Merge (reduce runs of equal labels) and Compress ----------------------------------------
__global__ void __launch_bounds__(OT) heads_kernel(const u64* __restrict__ keys, i64 n, int* __restrict__ head) {
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

__global__ void __launch_bounds__(OT) coo_pos_kernel(const u64* __restrict__ ukeys, i64 nnz, i64 m, i64 J, i64* __restrict__ pos) {
    for (i64 i = (i64)blockIdx.x * OT + threadIdx.x; i <= m; i += (i64)gridDim.x * OT) {
        const u64 want = (u64)i * (u64)J;
        i64 lo = 0, hi = nnz;
        while (lo < hi) {
            const i64 mid = (lo + hi) >> 1;
            if (ukeys[mid] < want) lo = mid + 1; else hi = mid;
        }
        pos[i] = lo;
    }
}

template <typename T>
__global__ void __launch_bounds__(OT) coo_out_kernel(const u64* __restrict__ ukeys, const T* __restrict__ uvals, i64 nnz, i64 J,
                                                     int* __restrict__ Ccrd, T* __restrict__ Cval) {
    for (i64 t = (i64)blockIdx.x * OT + threadIdx.x; t < nnz; t += (i64)gridDim.x * OT) {
        Ccrd[t] = (int)(ukeys[t] % (u64)J);
        Cval[t] = uvals[t];
    }
}

// ---- dense second-order workspace -------------------------------------------------------------
__global__ void __launch_bounds__(OT) dense2_count_kernel(const unsigned* __restrict__ bits, i64 m, i64 row_words, int* __restrict__ cnt) {
    const int lane = threadIdx.x & 31;
    for (i64 i = ((i64)blockIdx.x * OT + threadIdx.x) >> 5; i < m; i += ((i64)gridDim.x * OT) >> 5) {
        int c = 0;
        for (i64 w = lane; w < row_words; w += 32) c += __popc(bits[i * row_words + w]);
        for (int d = 16; d > 0; d >>= 1) c += __shfl_xor_sync(0xffffffffu, c, d);
        if (lane == 0) cnt[i] = c;
    }
}

// Copies a row's flagged positions out in column order.
template <typename T>
__global__ void __launch_bounds__(OT) dense2_emit_kernel(unsigned* __restrict__ bits, T* __restrict__ dvals, i64 m, i64 J, i64 row_words,
                                                         const i64* __restrict__ pos, int* __restrict__ Ccrd, T* __restrict__ Cval) {
    const int lane = threadIdx.x & 31;
    for (i64 i = ((i64)blockIdx.x * OT + threadIdx.x) >> 5; i < m; i += ((i64)gridDim.x * OT) >> 5) {
        i64 o = pos[i];
        if (pos[i + 1] == o) continue;
        for (i64 w0 = 0; w0 < row_words; w0 += 32) {
            const i64 w = w0 + lane;
            unsigned word = (w < row_words) ? bits[i * row_words + w] : 0u;
            const int pc = __popc(word);
            const int incl = warp_incl_scan(pc);
            i64 at = o + incl - pc;
            while (word) {
                const int b = __ffs(word) - 1;
                word &= word - 1;
                const i64 j = (w << 5) + b;
                Ccrd[at] = (int)j;
                Cval[at] = dvals[i * J + j];
                ++at;
            }
            o += __shfl_sync(0xffffffffu, incl, 31);
        }
    }
}

// ---- host side --------------------------------------------------------------------------------
static int grid_for(const LaunchCtx& c, i64 work_items, int per_block) {
    i64 want = (work_items + per_block - 1) / per_block;
    const i64 cap = (i64)c.sm_count * 16;
    if (want > cap) want = cap;
    return (int)(want < 1 ? 1 : want);
}

cudaError_t launch_outer_counts(const LaunchCtx& c, const Csr& At, const Csr& B, int* cnt) {
    if (At.nrows == 0) return cudaSuccess;
    outer_counts_kernel<<<grid_for(c, At.nrows, OT), OT, 0, c.stream>>>(At, B, cnt, c.ctl);
    ++c.launches;
    return cudaGetLastError();
}

// Sum over k of (entries of A's row k) x (entries of B's row k), added into a word the host can read.
__global__ void __launch_bounds__(OT) outer_total_kernel(Csr At, Csr B, u64* total) {
    i64 mine = 0;
    for (i64 k = (i64)blockIdx.x * OT + threadIdx.x; k < At.nrows; k += (i64)gridDim.x * OT)
        mine += (At.pos[k + 1] - At.pos[k]) * (B.pos[k + 1] - B.pos[k]);
    for (int d = 16; d > 0; d >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, d);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd_system(total, (u64)mine);
}

cudaError_t launch_outer_total(const LaunchCtx& c, const Csr& At, const Csr& B, u64* total_mapped_host) {
    if (At.nrows == 0) return cudaSuccess;
    outer_total_kernel<<<grid_for(c, At.nrows, OT), OT, 0, c.stream>>>(At, B, total_mapped_host);
    return cudaGetLastError();
}

size_t outer_sort_scratch_bytes(i64 n) {
    const i64 nblocks = (n + RS_TILE - 1) / RS_TILE;
    const size_t cells = (size_t)256 * (size_t)(nblocks > 0 ? nblocks : 1);
    return ((cells * 4 + 255) & ~(size_t)255) + (((cells + 1) * 8 + 255) & ~(size_t)255) + (((cells / 2048 + 2) * 8 + 255) & ~(size_t)255);
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
    if ((e = cudaMemcpyAsync(cnt_host_pinned, cnt_dev, sizeof(i64), cudaMemcpyDeviceToHost, c.stream)) != cudaSuccess) return e;
    if ((e = cudaStreamSynchronize(c.stream)) != cudaSuccess) return e;
    *result_in_first = !first;
    return cudaGetLastError();
}

// One pass of the sparse second-order workspace over all products, in rounds of `cap`
// (Algorithm 1: when the accumulation array is full it is sorted and reduced on its own, then
// united with the all array; the entry that found it full opens the next round).
// Buffers: two (label, value) arrays of N = P + (cap < P ? cap : 0) entries, head flags and
// their scan (N, N + 1), sort temporaries.  On return *result_first tells which array holds the
// duplicate-free result; its length is in *nnz_host_pinned.
template <typename T, bool VALUES>
static cudaError_t outer_ism_t(const LaunchCtx& c, const Csr& At, const Csr& B, const i64* koff, i64 P, i64 cap, i64 J, int label_bits,
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
        outer_expand_kernel<T, VALUES, false><<<grid_for(c, n_new, OT * 4), OT, 0, c.stream>>>(At, B, koff, t0, n_new, J, kc + n_all,
                                                                                                 VALUES ? vc + n_all : nullptr, nullptr, nullptr, 0, c.ctl);
        ++c.launches;
        // Sort + reduce of the accumulation array alone
        bool in_first = true;
        cudaError_t e = sort_reduce_t<T, VALUES>(c, n_new, label_bits, kc + n_all, VALUES ? vc + n_all : nullptr, ko + n_all,
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

cudaError_t launch_outer_ism(const LaunchCtx& c, bool numeric, const Csr& At, const Csr& B, const i64* koff, i64 P, i64 cap, i64 J,
                             int label_bits, u64* kA, void* vA, u64* kB, void* vB, int* head, i64* at, char* sort_tmp,
                             i64* block_sums, i64* nnz_dev, i64* nnz_host_pinned, bool* result_first) {
    if (!numeric)
        return outer_ism_t<double, false>(c, At, B, koff, P, cap, J, label_bits, kA, nullptr, kB, nullptr, head, at, sort_tmp, block_sums,
                                          nnz_dev, nnz_host_pinned, result_first);
    return c.is_f64 ? outer_ism_t<double, true>(c, At, B, koff, P, cap, J, label_bits, kA, (double*)vA, kB, (double*)vB, head, at, sort_tmp,
                                                block_sums, nnz_dev, nnz_host_pinned, result_first)
                    : outer_ism_t<float, true>(c, At, B, koff, P, cap, J, label_bits, kA, (float*)vA, kB, (float*)vB, head, at, sort_tmp,
                                               block_sums, nnz_dev, nnz_host_pinned, result_first);
}

cudaError_t launch_coo_pos(const LaunchCtx& c, const u64* ukeys, i64 nnz, i64 m, i64 J, i64* pos) {
    coo_pos_kernel<<<grid_for(c, m + 1, OT), OT, 0, c.stream>>>(ukeys, nnz, m, J, pos);
    ++c.launches;
    return cudaGetLastError();
}

cudaError_t launch_coo_out(const LaunchCtx& c, const u64* ukeys, const void* uvals, i64 nnz, i64 J, int* Ccrd, void* Cval) {
    if (nnz == 0) return cudaSuccess;
    if (c.is_f64) coo_out_kernel<double><<<grid_for(c, nnz, OT), OT, 0, c.stream>>>(ukeys, (const double*)uvals, nnz, J, Ccrd, (double*)Cval);
    else coo_out_kernel<float><<<grid_for(c, nnz, OT), OT, 0, c.stream>>>(ukeys, (const float*)uvals, nnz, J, Ccrd, (float*)Cval);
    ++c.launches;
    return cudaGetLastError();
}

// Dense second-order workspace.  symbolic: flags only, per-row counts into cnt.  numeric: values
// added in place (the value array must be clear on entry; the copy-out leaves the flags alone and
// the caller clears both arrays before the next use).
cudaError_t launch_outer_dense(const LaunchCtx& c, bool numeric, const Csr& At, const Csr& B, const i64* koff, i64 P, i64 m, i64 J,
                               unsigned* dbits, void* dvals, int* cnt, const i64* pos, int* Ccrd, void* Cval) {
    const i64 row_words = (J + 31) / 32;
    if (P > 0) {
        const int g = grid_for(c, P, OT * 4);
        if (!numeric)
            outer_expand_kernel<double, false, true><<<g, OT, 0, c.stream>>>(At, B, koff, 0, P, J, nullptr, nullptr, dbits, nullptr, row_words, c.ctl);
        else if (c.is_f64)
            outer_expand_kernel<double, true, true><<<g, OT, 0, c.stream>>>(At, B, koff, 0, P, J, nullptr, nullptr, dbits, (double*)dvals, row_words, c.ctl);
        else
            outer_expand_kernel<float, true, true><<<g, OT, 0, c.stream>>>(At, B, koff, 0, P, J, nullptr, nullptr, dbits, (float*)dvals, row_words, c.ctl);
        ++c.launches;
    }
    if (m == 0) return cudaGetLastError();
    if (!numeric) {
        dense2_count_kernel<<<grid_for(c, m * 32, OT), OT, 0, c.stream>>>(dbits, m, row_words, cnt);
    } else if (c.is_f64) {
        dense2_emit_kernel<double><<<grid_for(c, m * 32, OT), OT, 0, c.stream>>>(dbits, (double*)dvals, m, J, row_words, pos, Ccrd, (double*)Cval);
    } else {
        dense2_emit_kernel<float><<<grid_for(c, m * 32, OT), OT, 0, c.stream>>>(dbits, (float*)dvals, m, J, row_words, pos, Ccrd, (float*)Cval);
    }
    ++c.launches;
    return cudaGetLastError();
}

}  // namespace spws
