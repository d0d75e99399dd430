// Higher-order scatters with a sparse result in coordinate form (Sec. 7.3):
//   form 0  SpTTM     A(i,j,l) = sum_k  B(k,i,j) * C(k,l)           third-order workspace over (i,j,l)
//   form 1  SpTTM-I   A(k,j,l) = sum_i  B(k,i,j) * C(i,l)           workspace over (k,j,l)
//   form 2  SpMTTKRP  A(i,j)   = sum_kl B(k,l,i) * C(k,j) * D(l,j)  second-order workspace over (i,j)
// B is a CSF 3-tensor stored in the order its indices are written; C and D are CSR.  Every form
// walks B's stored entries; an entry meets the row of C its first (forms 0, 2) or second (form 1)
// coordinate picks, and the products are numbered entry by entry, C-row element by element.  The
// workspace is the sparse one of Algorithm 1 on integer labels (Sec. 5.2): the numbered products
// are appended in rounds of the accumulation array's capacity, sorted, reduced and united with
// the all array (sortmerge.cuh); the duplicate-free labels are then unpacked into coordinates.
// In form 2 a numbered product exists only when D's row holds the column too; the others carry the
// absent label.
#include "sortmerge.cuh"

namespace spws {

// entry -> its fibre (level 1), fibre -> its slice (level 0)
__global__ void __launch_bounds__(OT) csf_parents_kernel(Csf3Dev B, int* __restrict__ fib_of, int* __restrict__ slice_of) {
    const i64 stride = (i64)gridDim.x * OT;
    for (i64 f = (i64)blockIdx.x * OT + threadIdx.x; f < B.n1; f += stride)
        for (i64 e = B.pos2[f]; e < B.pos2[f + 1]; ++e) fib_of[e] = (int)f;
    const int lane = threadIdx.x & 31;
    for (i64 s = ((i64)blockIdx.x * OT + threadIdx.x) >> 5; s < B.n0; s += stride >> 5)
        for (i64 f = B.pos1[s] + lane; f < B.pos1[s + 1]; f += 32) slice_of[f] = (int)s;
}

// numbered products of entry e = length of the C row it picks
__global__ void __launch_bounds__(OT) higher_counts_kernel(int form, Csf3Dev B, Csr C, const int* __restrict__ fib_of,
                                                           const int* __restrict__ slice_of, int* __restrict__ cnt, DevCtl* ctl) {
    for (i64 e = (i64)blockIdx.x * OT + threadIdx.x; e < B.nnz; e += (i64)gridDim.x * OT) {
        const int f = fib_of[e];
        const int pick = form == 1 ? B.crd1[f] : B.crd0[slice_of[f]];
        int c = 0;
        if ((unsigned)pick < (unsigned)C.nrows) c = (int)(C.pos[pick + 1] - C.pos[pick]);
        else raise_status(ctl, DEV_NONCANONICAL);
        cnt[e] = c;
    }
}

__device__ __forceinline__ i64 owner_entry(const i64* __restrict__ eoff, i64 n, i64 t) {
    i64 lo = 0, hi = n;
    while (hi - lo > 1) {
        const i64 mid = (lo + hi) >> 1;
        if (eoff[mid] <= t) lo = mid; else hi = mid;
    }
    return lo;
}

// d1, d2: the extents the label is built from: label = (c_a * d1 + c_b) * d2 + c_c (forms 0, 1), c_a * d2 + c_b (form 2)
template <typename T, bool VALUES>
__global__ void __launch_bounds__(OT) higher_expand_kernel(int form, Csf3Dev B, Csr C, Csr D, const int* __restrict__ fib_of,
                                                           const int* __restrict__ slice_of, const i64* __restrict__ eoff, i64 t0, i64 n,
                                                           u64 d1, u64 d2, u64* __restrict__ keys, T* __restrict__ vals) {
    const T* __restrict__ Bval = (const T*)B.val;
    const T* __restrict__ Cval = (const T*)C.val;
    const T* __restrict__ Dval = (const T*)D.val;
    for (i64 s = ((i64)blockIdx.x * OT + threadIdx.x) * 4; s < n; s += (i64)gridDim.x * OT * 4) {
        i64 t = t0 + s;
        i64 e = owner_entry(eoff, B.nnz, t);
        for (int x = 0; x < 4 && s + x < n; ++x, ++t) {
            while (eoff[e + 1] <= t) ++e;
            const int f = fib_of[e];
            const int c0 = B.crd0[slice_of[f]], c1 = B.crd1[f], c2 = B.crd2[e];
            const i64 q = C.pos[form == 1 ? c1 : c0] + (t - eoff[e]);
            const int cc = C.crd[q];
            u64 label;
            T v = 0;
            if (form == 0) {            // (k,i,j) x C(k,l) -> (i,j,l)
                label = ((u64)c1 * d1 + (u64)c2) * d2 + (u64)cc;
                if (VALUES) v = mul_rn(Bval[e], Cval[q]);
            } else if (form == 1) {     // (k,i,j) x C(i,l) -> (k,j,l)
                label = ((u64)c0 * d1 + (u64)c2) * d2 + (u64)cc;
                if (VALUES) v = mul_rn(Bval[e], Cval[q]);
            } else {                    // (k,l,i) x C(k,j) x D(l,j) -> (i,j), when D's row l holds j
                label = ABSENT_LABEL;
                i64 lo = D.pos[c1], hi = D.pos[c1 + 1];
                while (lo < hi) {
                    const i64 mid = (lo + hi) >> 1;
                    if (D.crd[mid] < cc) lo = mid + 1; else hi = mid;
                }
                if (lo < D.pos[c1 + 1] && D.crd[lo] == cc) {
                    label = (u64)c2 * d2 + (u64)cc;
                    if (VALUES) v = mul_rn(mul_rn(Bval[e], Cval[q]), Dval[lo]);
                }
            }
            keys[s + x] = label;
            if (VALUES) vals[s + x] = v;
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(OT) higher_unpack_kernel(int order, const u64* __restrict__ ukeys, const T* __restrict__ uvals, i64 nnz,
                                                           u64 d1, u64 d2, int* __restrict__ o0, int* __restrict__ o1, int* __restrict__ o2,
                                                           T* __restrict__ oval) {
    for (i64 t = (i64)blockIdx.x * OT + threadIdx.x; t < nnz; t += (i64)gridDim.x * OT) {
        const u64 key = ukeys[t];
        if (order == 3) {
            o2[t] = (int)(key % d2);
            const u64 r = key / d2;
            o1[t] = (int)(r % d1);
            o0[t] = (int)(r / d1);
        } else {
            o1[t] = (int)(key % d2);
            o0[t] = (int)(key / d2);
        }
        oval[t] = uvals[t];
    }
}

// Number of numbered products, walking the tensor from its top level: a warp per stored level-0
// coordinate, lanes over its fibres; the total is added into a word the host can read.
__global__ void __launch_bounds__(OT) higher_total_kernel(int form, Csf3Dev B, Csr C, u64* total) {
    const int lane = threadIdx.x & 31;
    i64 mine = 0;
    for (i64 s = ((i64)blockIdx.x * OT + threadIdx.x) >> 5; s < B.n0; s += ((i64)gridDim.x * OT) >> 5) {
        const int c0 = B.crd0[s];
        for (i64 f = B.pos1[s] + lane; f < B.pos1[s + 1]; f += 32) {
            const int pick = form == 1 ? B.crd1[f] : c0;
            if ((unsigned)pick < (unsigned)C.nrows) mine += (B.pos2[f + 1] - B.pos2[f]) * (C.pos[pick + 1] - C.pos[pick]);
        }
    }
    for (int d = 16; d > 0; d >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, d);
    if (lane == 0 && mine) atomicAdd_system(total, (u64)mine);
}

// ---- host side --------------------------------------------------------------------------------
cudaError_t launch_higher_total(const LaunchCtx& c, int form, const Csf3Dev& B, const Csr& C, u64* total_mapped_host) {
    if (B.n0 == 0) return cudaSuccess;
    higher_total_kernel<<<grid_for(c, (i64)B.n0 * 32, OT), OT, 0, c.stream>>>(form, B, C, total_mapped_host);
    return cudaGetLastError();
}

cudaError_t launch_higher_setup(const LaunchCtx& c, int form, const Csf3Dev& B, const Csr& C, int* fib_of, int* slice_of, int* cnt) {
    if (B.nnz == 0) return cudaSuccess;
    csf_parents_kernel<<<grid_for(c, B.n1 > (i64)B.n0 * 32 ? B.n1 : (i64)B.n0 * 32, OT), OT, 0, c.stream>>>(B, fib_of, slice_of);
    higher_counts_kernel<<<grid_for(c, B.nnz, OT), OT, 0, c.stream>>>(form, B, C, fib_of, slice_of, cnt, c.ctl);
    c.launches += 2;
    return cudaGetLastError();
}

template <typename T, bool VALUES>
static cudaError_t higher_ism_t(const LaunchCtx& c, int form, const Csf3Dev& B, const Csr& C, const Csr& D, const int* fib_of,
                                const int* slice_of, const i64* eoff, i64 P, i64 cap, u64 d1, u64 d2, int label_bits, u64* kA, T* vA,
                                u64* kB, T* vB, int* head, i64* at, char* sort_tmp, i64* block_sums, i64* nnz_dev, i64* nnz_host_pinned,
                                bool* result_first) {
    auto expand = [&](i64 t0, i64 n, u64* keys, T* vals) -> cudaError_t {
        higher_expand_kernel<T, VALUES><<<grid_for(c, n, OT * 4), OT, 0, c.stream>>>(form, B, C, D, fib_of, slice_of, eoff, t0, n, d1, d2, keys, vals);
        ++c.launches;
        return cudaGetLastError();
    };
    return ism_rounds_t<T, VALUES>(c, expand, P, cap, label_bits, kA, vA, kB, vB, head, at, sort_tmp, block_sums, nnz_dev, nnz_host_pinned,
                                   result_first);
}

cudaError_t launch_higher_ism(const LaunchCtx& c, bool numeric, int form, const Csf3Dev& B, const Csr& C, const Csr& D, const int* fib_of,
                              const int* slice_of, const i64* eoff, i64 P, i64 cap, u64 d1, u64 d2, int label_bits, u64* kA, void* vA,
                              u64* kB, void* vB, int* head, i64* at, char* sort_tmp, i64* block_sums, i64* nnz_dev,
                              i64* nnz_host_pinned, bool* result_first) {
    if (!numeric)
        return higher_ism_t<double, false>(c, form, B, C, D, fib_of, slice_of, eoff, P, cap, d1, d2, label_bits, kA, nullptr, kB, nullptr, head,
                                           at, sort_tmp, block_sums, nnz_dev, nnz_host_pinned, result_first);
    return c.is_f64 ? higher_ism_t<double, true>(c, form, B, C, D, fib_of, slice_of, eoff, P, cap, d1, d2, label_bits, kA, (double*)vA, kB,
                                                 (double*)vB, head, at, sort_tmp, block_sums, nnz_dev, nnz_host_pinned, result_first)
                    : higher_ism_t<float, true>(c, form, B, C, D, fib_of, slice_of, eoff, P, cap, d1, d2, label_bits, kA, (float*)vA, kB,
                                                (float*)vB, head, at, sort_tmp, block_sums, nnz_dev, nnz_host_pinned, result_first);
}

cudaError_t launch_higher_unpack(const LaunchCtx& c, int order, const u64* ukeys, const void* uvals, i64 nnz, u64 d1, u64 d2, int* o0,
                                 int* o1, int* o2, void* oval) {
    if (nnz == 0) return cudaSuccess;
    if (c.is_f64)
        higher_unpack_kernel<double><<<grid_for(c, nnz, OT), OT, 0, c.stream>>>(order, ukeys, (const double*)uvals, nnz, d1, d2, o0, o1, o2, (double*)oval);
    else
        higher_unpack_kernel<float><<<grid_for(c, nnz, OT), OT, 0, c.stream>>>(order, ukeys, (const float*)uvals, nnz, d1, d2, o0, o1, o2, (float*)oval);
    ++c.launches;
    return cudaGetLastError();
}

}  // namespace spws
