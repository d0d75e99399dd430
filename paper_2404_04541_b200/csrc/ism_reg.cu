// Insert-sort-merge workspace held in registers: one group of G lanes per output row whose
// product count is at most G (Algorithm 1 with the accumulation array = the lanes of the group;
// coordinate-sort policy, Sec. 5.2: append without reduction, sort, reduce equal coordinates).
//   Insert : lane t takes the t-th product of the row in loop order (k, then j).
//   Sort   : bitonic network over the group on the packed word (j - jmin) << 5 | lane -- only
//            this integer moves (accumulation indexing, Sec. 5.1); values stay in their lane.
//   Merge  : equal coordinates are adjacent; the first lane of a run sums the run in product
//            order and writes it at row_ptr[i] + rank.
#include "common.cuh"

namespace spws {

template <typename T, int G, bool NUMERIC>
__global__ void __launch_bounds__(256) ism_reg_kernel(const int* __restrict__ perm, const DevCtl* __restrict__ ctl, int cls,
                                                      Csr A, Csr B, const int* __restrict__ jmin, int* __restrict__ cnt,
                                                      const i64* __restrict__ rowptr, int* __restrict__ Ccrd, T* __restrict__ Cval) {
    if (ctl->status != 0) return;
    int off, n;
    class_range(ctl, cls, off, n);
    const int* __restrict__ rows = perm + off;
    const unsigned lane = threadIdx.x & 31;
    const int gl = threadIdx.x % G;
    const unsigned gshift = lane - gl;
    const unsigned gmask = (G == 32) ? 0xffffffffu : (((1u << G) - 1u) << gshift);
    const i64 group = ((i64)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const i64 ngroups = ((i64)gridDim.x * blockDim.x) / G;
    const T* __restrict__ Aval = (const T*)A.val;
    const T* __restrict__ Bval = (const T*)B.val;

    // the row id and its A range are loaded one iteration ahead: with a handful of products per row
    // the kernel is a chain of dependent loads otherwise
    int row_n = 0;
    i64 ps_n = 0, pe_n = 0;
    if (group < n) {
        row_n = __ldg(rows + group);
        ps_n = __ldg(A.pos + row_n);
        pe_n = __ldg(A.pos + row_n + 1);
    }
    for (i64 r = group; r < n; r += ngroups) {
        const int row = row_n;
        const i64 ps = ps_n, pe = pe_n;
        if (r + ngroups < n) {
            row_n = __ldg(rows + r + ngroups);
            ps_n = __ldg(A.pos + row_n);
            pe_n = __ldg(A.pos + row_n + 1);
        }
        const int base = jmin[row];

        if (pe - ps == 1) {
            // A row with ONE entry (the commonest fibre of a hyper-sparse 3-tensor): its products
            // are the picked B row itself, already sorted and free of duplicates, so Insert, Sort
            // and Merge are the identity and the lanes copy the scaled B row to the output.
            const int k = __ldg(A.crd + ps);
            i64 qs = 0;
            int len = 0;
            if ((unsigned)k < (unsigned)B.nrows) {
                qs = __ldg(B.pos + k);
                len = min((int)(__ldg(B.pos + k + 1) - qs), G);
            }
            if (!NUMERIC) {
                if (gl == 0) cnt[row] = len;
            } else if (gl < len) {
                const i64 o = rowptr[row] + gl;
                Ccrd[o] = __ldg(B.crd + qs + gl);
                Cval[o] = mul_rn(__ldg(Aval + ps), __ldg(Bval + qs + gl));
            }
            continue;
        }

        // ---- Insert: lane gl receives product number gl
        unsigned packed = 0xffffffffu;
        T val = 0;
        int done = 0;
        for (i64 p0 = ps; p0 < pe; p0 += G) {
            const i64 p = p0 + gl;
            int len = 0;
            i64 qs = 0;
            if (p < pe) {
                const int k = __ldg(A.crd + p);
                if ((unsigned)k < (unsigned)B.nrows) {
                    qs = __ldg(B.pos + k);
                    len = (int)(__ldg(B.pos + k + 1) - qs);
                }
            }
            int incl = len;
#pragma unroll
            for (int d = 1; d < G; d <<= 1) {
                const int t = __shfl_up_sync(gmask, incl, d, G);
                if (gl >= d) incl += t;
            }
            const int excl = incl - len + done;
            const int total = __shfl_sync(gmask, incl, G - 1, G);
            // entry that owns product gl: the last entry whose first product is <= gl
            int e = 0;
#pragma unroll
            for (int s = G / 2; s >= 1; s >>= 1) {
                const int v = __shfl_sync(gmask, excl, e + s, G);
                if (v <= gl) e += s;
            }
            const int e_excl = __shfl_sync(gmask, excl, e, G);
            const i64 e_qs = __shfl_sync(gmask, qs, e, G);
            if (gl >= done && gl < done + total) {
                const i64 q = e_qs + (gl - e_excl);
                const int j = __ldg(B.crd + q);
                packed = ((unsigned)(j - base) << 5) | (unsigned)gl;
                if (NUMERIC) val = mul_rn(__ldg(Aval + p0 + e), __ldg(Bval + q));
            }
            done += total;
        }

        // ---- Sort
#pragma unroll
        for (int k = 2; k <= G; k <<= 1) {
#pragma unroll
            for (int j = k >> 1; j > 0; j >>= 1) {
                const unsigned other = __shfl_xor_sync(gmask, packed, j, G);
                const bool up = (gl & k) == 0;
                const bool low = (gl & j) == 0;
                packed = (up == low) ? min(packed, other) : max(packed, other);
            }
        }

        // ---- Merge
        const bool valid = packed != 0xffffffffu;
        const unsigned key = packed >> 5;
        const unsigned prev = __shfl_up_sync(gmask, key, 1, G);
        const bool head = valid && (gl == 0 || key != prev);
        const unsigned heads = (__ballot_sync(gmask, head) >> gshift) & ((G == 32) ? 0xffffffffu : ((1u << G) - 1u));
        if (!NUMERIC) {
            if (gl == 0) cnt[row] = __popc(heads);
        } else {
            T v = __shfl_sync(gmask, val, packed & 31u, G);
            T sum = v;
            for (int d = 1; d < G; ++d) {
                const unsigned k2 = __shfl_down_sync(gmask, key, d, G);
                const T v2 = __shfl_down_sync(gmask, v, d, G);
                const bool more = valid && (gl + d < G) && (k2 == key);
                if (!__any_sync(gmask, more)) break;
                if (more) sum = add_rn(sum, v2);
            }
            if (head) {
                const int rank = __popc(heads & ((1u << gl) - 1u));
                const i64 out = rowptr[row] + rank;
                Ccrd[out] = (int)key + base;
                Cval[out] = sum;
            }
        }
    }
}

// Rows with ONE A entry that picks a B row of at most 8 entries (the commonest fibre of a
// hyper-sparse 3-tensor): the products are the picked B row itself, already sorted and free of
// duplicates, so Insert, Sort and Merge are the identity and the row is copied out scaled.  Every
// lane first walks one row's chain of dependent loads (row id, A range, A entry, B range, output
// offset), 32 chains per warp in flight; then the warp copies the 32 rows together, eight lanes per
// row and four rows per step.
template <typename T>
__global__ void __launch_bounds__(256) copy_rows_kernel(const int* __restrict__ perm, const DevCtl* __restrict__ ctl, Csr A, Csr B,
                                                        const i64* __restrict__ rowptr, int* __restrict__ Ccrd, T* __restrict__ Cval) {
    if (ctl->status != 0) return;
    int off, n;
    class_range(ctl, CLS_COPY8, off, n);
    const int* __restrict__ rows = perm + off;
    const int lane = threadIdx.x & 31;
    const T* __restrict__ Aval = (const T*)A.val;
    const T* __restrict__ Bval = (const T*)B.val;
    const i64 stride = (i64)gridDim.x * blockDim.x;
    for (i64 r0 = ((i64)blockIdx.x * blockDim.x + threadIdx.x) - lane; r0 < n; r0 += stride) {
        const i64 r = r0 + lane;
        i64 qs = 0, out = 0;
        int len = 0;
        T a = 0;
        if (r < n) {
            const int row = __ldg(rows + r);
            const i64 p = __ldg(A.pos + row);
            const int k = __ldg(A.crd + p);
            a = __ldg(Aval + p);
            out = __ldg(rowptr + row);
            if ((unsigned)k < (unsigned)B.nrows) {
                qs = __ldg(B.pos + k);
                len = min((int)(__ldg(B.pos + k + 1) - qs), 8);
            }
        }
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            const int src = 4 * s + (lane >> 3), e = lane & 7;
            const i64 q = __shfl_sync(0xffffffffu, qs, src), o = __shfl_sync(0xffffffffu, out, src);
            const int l = __shfl_sync(0xffffffffu, len, src);
            const T av = __shfl_sync(0xffffffffu, a, src);
            if (e < l) {
                Ccrd[o + e] = __ldg(B.crd + q + e);
                Cval[o + e] = mul_rn(av, __ldg(Bval + q + e));
            }
        }
    }
}

template <typename T, int G>
static cudaError_t launch_g(const LaunchCtx& c, bool numeric, int cls, int n_host, const Csr& A, const Csr& B,
                            const i64* rowptr, int* Ccrd, void* Cval) {
    const int threads = 256;
    i64 groups = (n_host >= 0) ? n_host : A.nrows;
    i64 want = (groups * G + threads - 1) / threads;
    i64 cap = (i64)c.sm_count * 16;
    int grid = (int)(want < cap ? want : cap);
    if (grid < 1) grid = 1;
    if (numeric)
        ism_reg_kernel<T, G, true><<<grid, threads, 0, c.stream>>>(c.tab.perm, c.ctl, cls, A, B,
                                                                 c.tab.jmin, c.tab.cnt, rowptr, Ccrd, (T*)Cval);
    else
        ism_reg_kernel<T, G, false><<<grid, threads, 0, c.stream>>>(c.tab.perm, c.ctl, cls, A, B,
                                                                  c.tab.jmin, c.tab.cnt, rowptr, Ccrd, (T*)Cval);
    ++c.launches;
    return cudaGetLastError();
}

cudaError_t launch_ism_reg(const LaunchCtx& c, bool numeric, int cls, int n_host, const Csr& A, const Csr& B,
                           const i64* rowptr, int* Ccrd, void* Cval) {
    if (cls == CLS_COPY8 && numeric) {
        const i64 rows = n_host >= 0 ? n_host : A.nrows;
        i64 want = (rows + 255) / 256, cap = (i64)c.sm_count * 16;
        const int grid = (int)(want < 1 ? 1 : (want < cap ? want : cap));
        if (c.is_f64) copy_rows_kernel<double><<<grid, 256, 0, c.stream>>>(c.tab.perm, c.ctl, A, B, rowptr, Ccrd, (double*)Cval);
        else copy_rows_kernel<float><<<grid, 256, 0, c.stream>>>(c.tab.perm, c.ctl, A, B, rowptr, Ccrd, (float*)Cval);
        ++c.launches;
        return cudaGetLastError();
    }
    if (c.is_f64) {
        if (cls == CLS_ISM_REG8 || cls == CLS_COPY8) return launch_g<double, 8>(c, numeric, cls, n_host, A, B, rowptr, Ccrd, Cval);
        if (cls == CLS_ISM_REG16) return launch_g<double, 16>(c, numeric, cls, n_host, A, B, rowptr, Ccrd, Cval);
        return launch_g<double, 32>(c, numeric, cls, n_host, A, B, rowptr, Ccrd, Cval);
    }
    if (cls == CLS_ISM_REG8 || cls == CLS_COPY8) return launch_g<float, 8>(c, numeric, cls, n_host, A, B, rowptr, Ccrd, Cval);
    if (cls == CLS_ISM_REG16) return launch_g<float, 16>(c, numeric, cls, n_host, A, B, rowptr, Ccrd, Cval);
    return launch_g<float, 32>(c, numeric, cls, n_host, A, B, rowptr, Ccrd, Cval);
}

}  // namespace spws
