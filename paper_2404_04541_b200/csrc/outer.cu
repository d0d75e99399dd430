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
#include "sortmerge.cuh"

namespace spws {

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

template <typename T, bool VALUES>
static cudaError_t outer_ism_t(const LaunchCtx& c, const Csr& At, const Csr& B, const i64* koff, i64 P, i64 cap, i64 J, int label_bits,
                               u64* kA, T* vA, u64* kB, T* vB, int* head, i64* at, char* sort_tmp, i64* block_sums,
                               i64* nnz_dev, i64* nnz_host_pinned, bool* result_first) {
    auto expand = [&](i64 t0, i64 n, u64* keys, T* vals) -> cudaError_t {
        outer_expand_kernel<T, VALUES, false><<<grid_for(c, n, OT * 4), OT, 0, c.stream>>>(At, B, koff, t0, n, J, keys, vals, nullptr, nullptr, 0, c.ctl);
        ++c.launches;
        return cudaGetLastError();
    };
    return ism_rounds_t<T, VALUES>(c, expand, P, cap, label_bits, kA, vA, kB, vB, head, at, sort_tmp, block_sums, nnz_dev, nnz_host_pinned,
                                   result_first);
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
