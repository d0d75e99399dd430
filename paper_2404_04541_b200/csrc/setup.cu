// Symbolic-pass set-up kernels: input validation, per-row product upper bound and column
// span, routing of rows to workspaces (binning), exclusive scans, CSF level rebuild.
#include "common.cuh"

namespace spws {

// ---------------------------------------------------------------------------------------
// Validation: pos non-decreasing with pos[0] = 0 and pos[rows] = nnz; coordinates in range
// and strictly increasing inside a row.
// ---------------------------------------------------------------------------------------
__global__ void validate_csr_kernel(Csr M, i64 nnz, int coord_limit, DevCtl* ctl) {
    const i64 stride = (i64)gridDim.x * blockDim.x;
    bool bad = false;
    for (i64 r = (i64)blockIdx.x * blockDim.x + threadIdx.x; r < M.nrows; r += stride) {
        const i64 s = M.pos[r], e = M.pos[r + 1];
        if (r == 0 && s != 0) bad = true;
        if (r == M.nrows - 1 && e != nnz) bad = true;
        if (s > e || s < 0 || e > nnz) { bad = true; continue; }
        int prev = -1;
        for (i64 p = s; p < e; ++p) {
            const int c = M.crd[p];
            if (c <= prev || c >= coord_limit) bad = true;
            prev = c;
        }
    }
    if (M.nrows == 0 && threadIdx.x == 0 && blockIdx.x == 0 && nnz != 0) bad = true;
    if (bad) raise_status(ctl, DEV_NONCANONICAL);
}

cudaError_t launch_validate(const LaunchCtx& c, const Csr& A, const Csr& B, i64 nnzA, i64 nnzB) {
    const int grid = c.sm_count * 8;
    validate_csr_kernel<<<grid, 256, 0, c.stream>>>(A, nnzA, B.nrows, c.ctl);
    validate_csr_kernel<<<grid, 256, 0, c.stream>>>(B, nnzB, B.ncols, c.ctl);
    c.launches += 2;
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Per-row upper bound ub[i] = sum over A(i,:) of the picked B row's length, the exact span
// [jmin, jmax] of the candidate columns (first / last coordinate of the picked B rows, which
// are sorted), and the workspace class of the row.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ int dense_class(i64 ub, i64 span_words) {
    if (span_words <= DENSE_WARP_BM_WORDS && ub <= DENSE_WARP_MAX_UB) return CLS_DENSE_WARP;
    return ub >= DENSE_HUB_UB ? CLS_DENSE_HUB : CLS_DENSE_CTA;
}

__device__ __forceinline__ int classify_row(i64 ub, i64 entries, int jmin, int jmax, const ClassParams& prm, DevCtl* ctl) {
    if (ub == 0) return CLS_EMPTY;
    const i64 span = (i64)jmax - jmin + 1;
    const i64 span_words = (span + 31) >> 5;
    const bool dense_ok = span_words <= prm.max_span_words;
    const bool reg_ok = ub <= prm.reg_cap && span <= (1ll << 26);
    if (prm.policy == 0) {                       // dense forced
        if (!dense_ok) { raise_status(ctl, DEV_WORKSPACE_TOO_LARGE); return CLS_EMPTY; }
        return dense_class(ub, span_words);
    }
    // a single entry picking a short B row: Insert, Sort and Merge are the identity and the
    // output count is the B row's length, known right here
    const int reg_cls = ub <= 8 ? (entries == 1 ? CLS_COPY8 : CLS_ISM_REG8) : (ub <= 16 ? CLS_ISM_REG16 : CLS_ISM_REG);
    if (prm.policy == 1) {                       // sparse ISM forced
        if (reg_ok) return reg_cls;
        if (ub <= prm.smem_small_cap) return CLS_ISM_SMEM_S;
        if (ub <= prm.smem_cap) return CLS_ISM_SMEM;
        return CLS_ISM_GLOBAL;
    }
    if (prm.policy == 3) {                       // hash forced
        if (ub <= HASH_SMALL_CAP) return CLS_HASH_S;
        if (ub <= HASH_CAP) return CLS_HASH;
        return CLS_ISM_GLOBAL;
    }
    // auto: few products -> sort them in registers; a bitmap that is small next to the work ->
    // dense; mid-size rows -> shared-memory ISM; long rows -> dense; otherwise global ISM.
    if (reg_ok) return reg_cls;
    if (dense_ok && (float)span_words <= prm.span_words_per_product * (float)ub) return dense_class(ub, span_words);
    if (ub <= prm.smem_small_cap) return CLS_ISM_SMEM_S;
    if (ub <= prm.smem_cap) return CLS_ISM_SMEM;
    if (dense_ok) return dense_class(ub, span_words);
    return CLS_ISM_GLOBAL;
}

// First column, last column and length of every B row, in one 16-byte record: when A has several
// times more entries than B has rows, the bounds kernel reads the record of the row an entry picks
// (one load, neighbouring rows share sectors) instead of two offsets and two coordinates.
__global__ void __launch_bounds__(256) brow_summary_kernel(Csr B, int4* __restrict__ brow) {
    for (i64 k = (i64)blockIdx.x * blockDim.x + threadIdx.x; k < B.nrows; k += (i64)gridDim.x * blockDim.x) {
        const i64 qs = B.pos[k], qe = B.pos[k + 1];
        int4 s = make_int4(0x7fffffff, -1, 0, 0);
        if (qe > qs) {
            s.x = __ldg(B.crd + qs);
            s.y = __ldg(B.crd + qe - 1);
            s.z = (int)min(qe - qs, (i64)0x7fffffff);
        }
        brow[k] = s;
    }
}

// SUMMARY: brow holds the B-row summaries (the instantiation without them carries B's own arrays'
// two-level gathers and needs more registers).
template <int G, bool SUMMARY>
__global__ void __launch_bounds__(256) row_bounds_kernel(Csr A, Csr B, RowTables tab, ClassParams prm, DevCtl* ctl,
                                                         const int4* __restrict__ brow) {
    // rows and products per class, one histogram per warp: 64-bit shared-memory adds are
    // compare-and-swap loops, which many threads on one address turn into a queue
    __shared__ int s_hist[8][NCLASS];
    __shared__ i64 s_cprod[8][NCLASS];
    __shared__ i64 s_products, s_max_ub, s_max_ub_global, s_max_ub_smem;
    __shared__ int s_max_span_words;
    for (int x = threadIdx.x; x < 8 * NCLASS; x += blockDim.x) { (&s_hist[0][0])[x] = 0; (&s_cprod[0][0])[x] = 0; }
    if (threadIdx.x == 0) { s_products = 0; s_max_ub = 0; s_max_ub_global = 0; s_max_ub_smem = 0; s_max_span_words = 0; }
    __syncthreads();
    int* const w_hist = s_hist[threadIdx.x >> 5];
    i64* const w_cprod = s_cprod[threadIdx.x >> 5];
    const int gl = threadIdx.x % G;
    const unsigned lane = threadIdx.x & 31;
    const unsigned gmask = (G == 32) ? 0xffffffffu : (((1u << G) - 1u) << (lane - gl));
    const i64 group = ((i64)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const i64 ngroups = ((i64)gridDim.x * blockDim.x) / G;
    i64 my_products = 0, my_max = 0;
    // rows and products of the class of this group's last rows: neighbouring rows mostly share a
    // class, so the shared-memory histogram is touched only when the class changes
    int run_cls = -1, run_rows = 0, my_span_words = 0;
    i64 run_products = 0;
    for (i64 row = group; row < A.nrows; row += ngroups) {
        const i64 ps = A.pos[row], pe = A.pos[row + 1];
        if (pe - ps > LONG_A_ROW) {
            // a very long row would be this group's serial chain and set the kernel's time on power-law
            // inputs: it is listed for the kernel that gives such rows a CTA each (the list borrows the
            // table of warp rows, which is not in use before the numeric routing)
            if (gl == 0) tab.warp_rows[atomicAdd(&ctl->n_long_a, 1)] = (int)row;
            continue;
        }
        i64 u = 0;
        int lo = 0x7fffffff, hi = -1;
        bool bad = false;
        // four entries per lane and step, each level of loads issued for all four before the
        // next level needs it: a row with very many entries is a chain of dependent loads otherwise
        i64 p0 = ps + gl;
        if (pe - ps <= G) {                         // the common short row: one entry per lane
            if (p0 < pe) {
                const int k = __ldg(A.crd + p0);
                if ((unsigned)k < (unsigned)B.nrows) {
                    if (SUMMARY) {
                        const int4 s = __ldg(brow + k);
                        u = s.z;
                        lo = s.x;
                        hi = s.y;
                    } else {
                        const i64 qs = __ldg(B.pos + k), qe = __ldg(B.pos + k + 1);
                        if (qe > qs) {
                            u = qe - qs;
                            lo = __ldg(B.crd + qs);
                            hi = __ldg(B.crd + qe - 1);
                        }
                    }
                } else {
                    bad = true;
                }
            }
            p0 = pe;
        }
        for (; p0 < pe; p0 += 4 * G) {
            int k[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const i64 p = p0 + (i64)x * G;
                k[x] = p < pe ? __ldg(A.crd + p) : -1;
                if (p < pe && (unsigned)k[x] >= (unsigned)B.nrows) bad = true;
            }
            if (SUMMARY) {
#pragma unroll
                for (int x = 0; x < 4; ++x)
                    if ((unsigned)k[x] < (unsigned)B.nrows) {
                        const int4 s = __ldg(brow + k[x]);
                        u += s.z;
                        lo = min(lo, s.x);
                        hi = max(hi, s.y);
                    }
                continue;
            }
            i64 qs[4], qe[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                qs[x] = qe[x] = 0;
                if ((unsigned)k[x] < (unsigned)B.nrows) { qs[x] = __ldg(B.pos + k[x]); qe[x] = __ldg(B.pos + k[x] + 1); }
            }
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                if (qe[x] > qs[x]) {
                    u += qe[x] - qs[x];
                    lo = min(lo, __ldg(B.crd + qs[x]));
                    hi = max(hi, __ldg(B.crd + qe[x] - 1));
                }
            }
        }
#pragma unroll
        for (int d = G / 2; d > 0; d >>= 1) {
            u += __shfl_xor_sync(gmask, u, d, G);
            lo = min(lo, __shfl_xor_sync(gmask, lo, d, G));
            hi = max(hi, __shfl_xor_sync(gmask, hi, d, G));
        }
        if (bad) raise_status(ctl, DEV_NONCANONICAL);
        if (gl == 0) {
            if (lo < 0 || hi >= B.ncols) { raise_status(ctl, DEV_NONCANONICAL); u = 0; }
            if (u > 0) lo &= ~31;               // bitmap words of every row start at a multiple of 32 columns
            const int cls = classify_row(u, pe - ps, lo, hi, prm, ctl);
            tab.ub[row] = u;
            tab.jmin[row] = lo;
            tab.jmax[row] = hi;
            tab.cnt[row] = cls == CLS_COPY8 ? (int)u : 0;
            tab.cls[row] = (unsigned char)cls;
            if (cls != run_cls) {
                if (run_rows) {
                    atomicAdd(&w_hist[run_cls], run_rows);
                    if (run_products) atomicAdd((u64*)&w_cprod[run_cls], (u64)run_products);
                }
                run_cls = cls;
                run_rows = 0;
                run_products = 0;
            }
            ++run_rows;
            run_products += u;
            my_products += u;
            my_max = max(my_max, u);
            // (rare classes: straight to shared memory, and only when the maximum would move)
            if (cls == CLS_ISM_GLOBAL && u > s_max_ub_global) atomicMax(&s_max_ub_global, u);
            if (cls == CLS_ISM_SMEM && u > s_max_ub_smem) atomicMax(&s_max_ub_smem, u);
            if (cls == CLS_DENSE_HUB || cls == CLS_DENSE_CTA || cls == CLS_DENSE_WARP)
                my_span_words = max(my_span_words, (hi - lo) / 32 + 1);
        }
    }
    if (gl == 0 && run_rows) {
        atomicAdd(&w_hist[run_cls], run_rows);
        if (run_products) atomicAdd((u64*)&w_cprod[run_cls], (u64)run_products);
    }
    // the totals: reduced over the warp first (lanes other than a group's first hold zeros)
    for (int d = 16; d > 0; d >>= 1) {
        my_products += __shfl_xor_sync(0xffffffffu, my_products, d);
        my_max = max(my_max, __shfl_xor_sync(0xffffffffu, my_max, d));
        my_span_words = max(my_span_words, __shfl_xor_sync(0xffffffffu, my_span_words, d));
    }
    if (lane == 0) {
        if (my_span_words) atomicMax(&s_max_span_words, my_span_words);
        if (my_products) atomicAdd((u64*)&s_products, (u64)my_products);
        if (my_max) atomicMax(&s_max_ub, my_max);
    }
    __syncthreads();
    if (threadIdx.x < NCLASS) {
        int rows = 0;
        i64 prods = 0;
        for (int w = 0; w < 8; ++w) { rows += s_hist[w][threadIdx.x]; prods += s_cprod[w][threadIdx.x]; }
        if (rows) atomicAdd(&ctl->class_count[threadIdx.x], rows);
        if (prods) atomicAdd((u64*)&ctl->class_products[threadIdx.x], (u64)prods);
    }
    if (threadIdx.x == 0) {
        if (s_products) atomicAdd((u64*)&ctl->products, (u64)s_products);
        if (s_max_ub) atomicMax(&ctl->max_ub, s_max_ub);
        if (s_max_ub_global) atomicMax(&ctl->max_ub_global, s_max_ub_global);
        if (s_max_ub_smem) atomicMax(&ctl->max_ub_smem, s_max_ub_smem);
        if (s_max_span_words) atomicMax(&ctl->max_span_words, s_max_span_words);
    }
}

// Bounds and class of the listed long rows, a CTA per row: 256 lanes across the entries, four
// entries per lane and step.
template <bool SUMMARY>
__global__ void __launch_bounds__(256) row_bounds_long_kernel(Csr A, Csr B, RowTables tab, ClassParams prm, DevCtl* ctl,
                                                              const int4* __restrict__ brow) {
    __shared__ i64 s_u[8];
    __shared__ int s_lo[8], s_hi[8], s_bad[8];
    const int n = min(ctl->n_long_a, A.nrows);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int r = blockIdx.x; r < n; r += gridDim.x) {
        const int row = tab.warp_rows[r];
        const i64 ps = A.pos[row], pe = A.pos[row + 1];
        i64 u = 0;
        int lo = 0x7fffffff, hi = -1, bad = 0;
        for (i64 p0 = ps + tid; p0 < pe; p0 += 4 * 256) {
            int k[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const i64 p = p0 + (i64)x * 256;
                k[x] = p < pe ? __ldg(A.crd + p) : -1;
                if (p < pe && (unsigned)k[x] >= (unsigned)B.nrows) bad = 1;
            }
            if (SUMMARY) {
                int4 s[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) s[x] = (unsigned)k[x] < (unsigned)B.nrows ? __ldg(brow + k[x]) : make_int4(0x7fffffff, -1, 0, 0);
#pragma unroll
                for (int x = 0; x < 4; ++x) { u += s[x].z; lo = min(lo, s[x].x); hi = max(hi, s[x].y); }
            } else {
                i64 qs[4], qe[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    qs[x] = qe[x] = 0;
                    if ((unsigned)k[x] < (unsigned)B.nrows) { qs[x] = __ldg(B.pos + k[x]); qe[x] = __ldg(B.pos + k[x] + 1); }
                }
#pragma unroll
                for (int x = 0; x < 4; ++x)
                    if (qe[x] > qs[x]) {
                        u += qe[x] - qs[x];
                        lo = min(lo, __ldg(B.crd + qs[x]));
                        hi = max(hi, __ldg(B.crd + qe[x] - 1));
                    }
            }
        }
        for (int d = 16; d > 0; d >>= 1) {
            u += __shfl_xor_sync(0xffffffffu, u, d);
            lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, d));
            hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, d));
            bad |= __shfl_xor_sync(0xffffffffu, bad, d);
        }
        __syncthreads();                                   // the previous row's totals have been read
        if (lane == 0) { s_u[warp] = u; s_lo[warp] = lo; s_hi[warp] = hi; s_bad[warp] = bad; }
        __syncthreads();
        if (tid == 0) {
            for (int w = 1; w < 8; ++w) { u += s_u[w]; lo = min(lo, s_lo[w]); hi = max(hi, s_hi[w]); bad |= s_bad[w]; }
            if (bad) raise_status(ctl, DEV_NONCANONICAL);
            if (lo < 0 || hi >= B.ncols) { raise_status(ctl, DEV_NONCANONICAL); u = 0; }
            if (u > 0) lo &= ~31;
            const int cls = classify_row(u, pe - ps, lo, hi, prm, ctl);
            tab.ub[row] = u;
            tab.jmin[row] = lo;
            tab.jmax[row] = hi;
            tab.cnt[row] = cls == CLS_COPY8 ? (int)u : 0;
            tab.cls[row] = (unsigned char)cls;
            atomicAdd(&ctl->class_count[cls], 1);
            if (u) {
                atomicAdd((u64*)&ctl->class_products[cls], (u64)u);
                atomicAdd((u64*)&ctl->products, (u64)u);
                atomicMax(&ctl->max_ub, u);
                if (cls == CLS_ISM_GLOBAL) atomicMax(&ctl->max_ub_global, u);
                if (cls == CLS_ISM_SMEM) atomicMax(&ctl->max_ub_smem, u);
                if (cls == CLS_DENSE_HUB || cls == CLS_DENSE_CTA || cls == CLS_DENSE_WARP)
                    atomicMax(&ctl->max_span_words, (hi - lo) / 32 + 1);
            }
        }
    }
}

cudaError_t launch_row_bounds(const LaunchCtx& c, const Csr& A, const Csr& B, i64 nnzA) {
    if (A.nrows == 0) return cudaSuccess;
    const double avg = (double)nnzA / (double)A.nrows;
    const int threads = 256;
    auto grid_for = [&](int G) {
        i64 want = ((i64)A.nrows * G + threads - 1) / threads;
        i64 cap = (i64)c.sm_count * 16;
        return (int)(want < cap ? want : cap);
    };
    // (one and two lanes per row were measured on the fibre matrix of the 3-tensor workload, 1.06
    // entries per row: slower than four)
    if (c.brow) {
        i64 want = ((i64)B.nrows + threads - 1) / threads;
        i64 cap = (i64)c.sm_count * 8;
        brow_summary_kernel<<<(int)(want < cap ? want : cap), threads, 0, c.stream>>>(B, c.brow);
        ++c.launches;
    }
    auto launch = [&](auto kernel, int G) { kernel<<<grid_for(G), threads, 0, c.stream>>>(A, B, c.tab, c.prm, c.ctl, c.brow); };
    const bool sm = c.brow != nullptr;
    if (avg <= 1.5) sm ? launch(row_bounds_kernel<1, true>, 1) : launch(row_bounds_kernel<1, false>, 1);
    else if (avg <= 3.0) sm ? launch(row_bounds_kernel<2, true>, 2) : launch(row_bounds_kernel<2, false>, 2);
    else if (avg <= 6.0) sm ? launch(row_bounds_kernel<4, true>, 4) : launch(row_bounds_kernel<4, false>, 4);
    else if (avg <= 12.0) sm ? launch(row_bounds_kernel<8, true>, 8) : launch(row_bounds_kernel<8, false>, 8);
    else sm ? launch(row_bounds_kernel<32, true>, 32) : launch(row_bounds_kernel<32, false>, 32);
    ++c.launches;
    // rows the kernel above listed as too long for a lane group (none, unless A has more than
    // LONG_A_ROW entries in all)
    if (nnzA > LONG_A_ROW) {
        const i64 most = nnzA / LONG_A_ROW;
        const int grid = (int)(most < (i64)c.sm_count * 4 ? most : (i64)c.sm_count * 4);
        if (sm) row_bounds_long_kernel<true><<<grid, 256, 0, c.stream>>>(A, B, c.tab, c.prm, c.ctl, c.brow);
        else row_bounds_long_kernel<false><<<grid, 256, 0, c.stream>>>(A, B, c.tab, c.prm, c.ctl, c.brow);
        ++c.launches;
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Word lists of long B rows.  The list of row k lives in `bw` at the positions of the row's own
// entries: bw[pos[k]] is a header (.x = number of pairs, 0 = no list), the pairs (.x = column / 32,
// .y = the bits of the row's entries in that word) follow.  A list is kept only when it has at
// most three quarters as many pairs as the row has entries.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) bw_find_long_kernel(Csr B, int* __restrict__ bw_long, int cap, DevCtl* ctl) {
    for (i64 k = (i64)blockIdx.x * blockDim.x + threadIdx.x; k < B.nrows; k += (i64)gridDim.x * blockDim.x) {
        if (B.pos[k + 1] - B.pos[k] >= BW_MIN_LEN) {
            const int at = atomicAdd(&ctl->n_long, 1);
            if (at < cap) bw_long[at] = (int)k;
        }
    }
}

constexpr int BWB_THREADS = 256;
constexpr int BWB_ITEMS = 4;

__global__ void __launch_bounds__(BWB_THREADS) bw_build_kernel(Csr B, const int* __restrict__ bw_long, int cap,
                                                              uint2* __restrict__ bw, DevCtl* ctl) {
    __shared__ int ws[33];
    __shared__ int s_next;
    const int n_long = min(ctl->n_long, cap);
    const int tid = threadIdx.x;
    for (;;) {
        __syncthreads();
        if (tid == 0) s_next = atomicAdd(&ctl->work_counter[BW_SLOT], 1);
        __syncthreads();
        if (s_next >= n_long) break;
        const int k = bw_long[s_next];
        const i64 qs = B.pos[k], qe = B.pos[k + 1];
        const i64 len = qe - qs;
        const int* __restrict__ crd = B.crd;
        int carry = 0;                                   // pairs of the row before this tile
        for (i64 t0 = qs; t0 < qe; t0 += BWB_THREADS * BWB_ITEMS) {
            const i64 q0 = t0 + (i64)tid * BWB_ITEMS;
            unsigned word[BWB_ITEMS], bits[BWB_ITEMS];
            int nfirst = 0;
            unsigned prev = (q0 > qs && q0 < qe) ? ((unsigned)__ldg(crd + q0 - 1) >> 5) : 0xffffffffu;
#pragma unroll
            for (int x = 0; x < BWB_ITEMS; ++x) {
                const i64 q = q0 + x;
                word[x] = 0xffffffffu;                   // not the first entry of a word
                bits[x] = 0u;
                if (q < qe) {
                    const unsigned c = (unsigned)__ldg(crd + q);
                    if ((c >> 5) != prev) {
                        word[x] = c >> 5;
                        unsigned b = 1u << (c & 31);
                        for (i64 q2 = q + 1; q2 < qe; ++q2) {          // at most 31 more entries share the word
                            const unsigned c2 = (unsigned)__ldg(crd + q2);
                            if ((c2 >> 5) != word[x]) break;
                            b |= 1u << (c2 & 31);
                        }
                        bits[x] = b;
                        ++nfirst;
                    }
                    prev = c >> 5;
                }
            }
            int total;
            int at = carry + block_excl_scan<BWB_THREADS>(nfirst, ws, total);
#pragma unroll
            for (int x = 0; x < BWB_ITEMS; ++x)
                if (word[x] != 0xffffffffu) {
                    if (at + 1 < len) bw[qs + 1 + at] = make_uint2(word[x], bits[x]);
                    ++at;
                }
            carry += total;
        }
        if (tid == 0) bw[qs] = make_uint2(4 * (i64)carry <= 3 * len ? (unsigned)carry : 0u, 0u);
    }
}

cudaError_t launch_bw_build(const LaunchCtx& c, const Csr& B) {
    if (!c.bw || B.nrows == 0) return cudaSuccess;
    i64 want = ((i64)B.nrows + 255) / 256;
    i64 cap = (i64)c.sm_count * 8;
    bw_find_long_kernel<<<(int)(want < cap ? want : cap), 256, 0, c.stream>>>(B, c.bw_long, c.bw_long_cap, c.ctl);
    bw_build_kernel<<<c.sm_count * 8, BWB_THREADS, 0, c.stream>>>(B, c.bw_long, c.bw_long_cap, c.bw, c.ctl);
    c.launches += 2;
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Binning: rows grouped by class into perm (class c occupies [off[c], off[c+1])); dense rows
// also reserve the slot of their occupancy bitmap in the arena.  Order inside a class follows
// block arrival.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) bin_rows_kernel(int m, RowTables tab, ClassParams prm, DevCtl* ctl) {
    __shared__ int s_hist[NCLASS], s_base[NCLASS], s_off[NCLASS];
    __shared__ int ws[33];
    __shared__ u64 s_bm_base;
    const int rows_per_block = blockDim.x * 4;
    if (threadIdx.x == 0) {
        int o = 0;
        for (int c = 0; c < NCLASS; ++c) { s_off[c] = o; o += ctl->class_count[c]; }
    }
    for (i64 r0 = (i64)blockIdx.x * rows_per_block; r0 < m; r0 += (i64)gridDim.x * rows_per_block) {
        if (threadIdx.x < NCLASS) s_hist[threadIdx.x] = 0;
        __syncthreads();
        int cls[4], rank[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const i64 row = r0 + x * blockDim.x + threadIdx.x;
            cls[x] = -1;
            if (row < m) {
                cls[x] = tab.cls[row];
                rank[x] = atomicAdd(&s_hist[cls[x]], 1);
            }
        }
        __syncthreads();
        if (threadIdx.x < NCLASS && s_hist[threadIdx.x])
            s_base[threadIdx.x] = atomicAdd(&ctl->class_cursor[threadIdx.x], s_hist[threadIdx.x]);
        __syncthreads();
        // bitmap words of this thread's dense rows; one arena reservation per block
        int words[4], my_words = 0;
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const i64 row = r0 + x * blockDim.x + threadIdx.x;
            words[x] = 0;
            if (cls[x] == CLS_DENSE_WARP || cls[x] == CLS_DENSE_HUB || cls[x] == CLS_DENSE_CTA)
            {   // the row's slot: bitmap words, then the rank at the start of every 32-word chunk
                const int nw = (tab.jmax[row] - tab.jmin[row]) / 32 + 1;
                words[x] = (nw + (nw + 31) / 32 + 3) & ~3;      // 16-byte aligned slots
            }
            my_words += words[x];
        }
        int block_words;
        int my_off = block_excl_scan<256>(my_words, ws, block_words);
        if (threadIdx.x == 0 && block_words) s_bm_base = atomicAdd(&ctl->bm_words_used, (u64)block_words);
        __syncthreads();
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const i64 row = r0 + x * blockDim.x + threadIdx.x;
            if (cls[x] < 0) continue;
            tab.perm[s_off[cls[x]] + s_base[cls[x]] + rank[x]] = (int)row;
            if (words[x]) {
                const u64 at = s_bm_base + (u64)my_off;
                my_off += words[x];
                if (at + (u64)words[x] > prm.bm_arena_words) {
                    raise_status(ctl, DEV_SCRATCH_TOO_SMALL);
                    tab.bm_off[row] = -1;
                } else {
                    tab.bm_off[row] = (i64)at;
                }
            }
        }
        __syncthreads();
    }
}

cudaError_t launch_bin_rows(const LaunchCtx& c, int m) {
    if (m == 0) return cudaSuccess;
    i64 want = ((i64)m + 1023) / 1024;
    i64 cap = (i64)c.sm_count * 8;
    bin_rows_kernel<<<(int)(want < cap ? want : cap), 256, 0, c.stream>>>(m, c.tab, c.prm, c.ctl);
    ++c.launches;
    return cudaGetLastError();
}

// Numeric routing of the dense rows, once their output counts are known: a row the warp kernel
// counted and whose outputs fit a warp's accumulator stays with a warp; every other row becomes
// one CTA unit, or several when it has many products: unit c of n takes the c-th n-th of the
// row's A entries (all units of a row add into the same outputs).
__global__ void __launch_bounds__(256) dense_rebin_kernel(int m, RowTables tab, ClassParams prm, DevCtl* ctl) {
    __shared__ int ws[33];
    __shared__ int s_wbase, s_ubase, s_wmax;
    __shared__ i64 s_wp, s_wn;
    int off, n4, n5, n6, o5, o6;
    class_range(ctl, CLS_DENSE_WARP, off, n4);
    class_range(ctl, CLS_DENSE_HUB, o5, n5);
    class_range(ctl, CLS_DENSE_CTA, o6, n6);
    const int n = n4 + n5 + n6;                       // the three classes are adjacent in perm
    const i64 unit_products = dense_unit_products(ctl->products);
    for (i64 b0 = (i64)blockIdx.x * blockDim.x; b0 < n; b0 += (i64)gridDim.x * blockDim.x) {
        const i64 r = b0 + threadIdx.x;
        int row = -1, cnt = 0, to_warp = 0, nu = 0;
        if (threadIdx.x == 0) { s_wp = 0; s_wn = 0; s_wmax = 0; }
        if (r < n) {
            row = tab.perm[off + r];
            cnt = tab.cnt[row];
            to_warp = tab.cls[row] == CLS_DENSE_WARP && cnt <= DENSE_WARP_ACC;
            nu = to_warp ? 0 : dense_units_of_row(tab.ub[row], unit_products);
        }
        int wtot, utot;
        const int wpos = block_excl_scan<256>(to_warp, ws, wtot);
        const int upos = block_excl_scan<256>(nu, ws, utot);
        if (threadIdx.x == 0) {
            s_wbase = wtot ? atomicAdd(&ctl->n_warp_rows, wtot) : 0;
            s_ubase = utot ? atomicAdd(&ctl->n_units, utot) : 0;
        }
        __syncthreads();
        if (row >= 0) {
            if (to_warp) {
                tab.warp_rows[s_wbase + wpos] = row;
                tab.row_unit0[row] = -1;
            } else {
                const int u0 = s_ubase + upos;
                if (u0 + nu > prm.unit_cap) {
                    raise_status(ctl, DEV_SCRATCH_TOO_SMALL);
                    tab.row_unit0[row] = -1;
                } else {
                    tab.row_unit0[row] = u0;
                    for (int t = 0; t < nu; ++t) tab.unit_row[u0 + t] = row;
                }
            }
        }
        {
            // products, outputs and largest output count of the warp rows: one shared atomic per warp
            i64 wp = (row >= 0 && to_warp) ? tab.ub[row] : 0;
            i64 wn = (row >= 0 && to_warp) ? cnt : 0;
            int wm = (row >= 0 && to_warp) ? cnt : 0;
            for (int d = 16; d > 0; d >>= 1) {
                wp += __shfl_xor_sync(0xffffffffu, wp, d);
                wn += __shfl_xor_sync(0xffffffffu, wn, d);
                wm = max(wm, __shfl_xor_sync(0xffffffffu, wm, d));
            }
            if ((threadIdx.x & 31) == 0 && wp) {
                atomicAdd((u64*)&s_wp, (u64)wp);
                atomicAdd((u64*)&s_wn, (u64)wn);
                atomicMax(&s_wmax, wm);
            }
        }
        __syncthreads();
        if (threadIdx.x == 0 && s_wp) {
            atomicAdd((u64*)&ctl->dense_warp_products, (u64)s_wp);
            atomicAdd((u64*)&ctl->dense_warp_nnz, (u64)s_wn);
            atomicMax(&ctl->max_warp_cnt, s_wmax);
        }
        __syncthreads();
    }
}

cudaError_t launch_dense_rebin(const LaunchCtx& c, int m, const i64* rowptr) {
    (void)rowptr;
    if (m == 0) return cudaSuccess;
    i64 want = ((i64)m + 255) / 256;
    i64 cap = (i64)c.sm_count * 8;
    dense_rebin_kernel<<<(int)(want < cap ? want : cap), 256, 0, c.stream>>>(m, c.tab, c.prm, c.ctl);
    ++c.launches;
    return cudaGetLastError();
}

// Output entries per class (statistics for the per-kernel byte counts): one pass over the rows in
// row order, every thread keeping a sum per class.
__global__ void __launch_bounds__(256) class_nnz_kernel(int m, RowTables tab, DevCtl* ctl) {
    i64 sum[NCLASS];
#pragma unroll
    for (int k = 0; k < NCLASS; ++k) sum[k] = 0;
    for (i64 row = (i64)blockIdx.x * blockDim.x + threadIdx.x; row < m; row += (i64)gridDim.x * blockDim.x) {
        const int c = tab.cls[row];
        const int v = tab.cnt[row];
#pragma unroll
        for (int k = 0; k < NCLASS; ++k) sum[k] += (c == k) ? v : 0;
    }
    __shared__ i64 s_part[8][NCLASS];
#pragma unroll
    for (int k = 0; k < NCLASS; ++k) {
        i64 t = sum[k];
        for (int d = 16; d > 0; d >>= 1) t += __shfl_xor_sync(0xffffffffu, t, d);
        if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5][k] = t;
    }
    __syncthreads();
    if (threadIdx.x < NCLASS && threadIdx.x != CLS_EMPTY) {
        i64 t = 0;
        for (int w = 0; w < 8; ++w) t += s_part[w][threadIdx.x];
        if (t) atomicAdd((u64*)&ctl->class_nnz[threadIdx.x], (u64)t);
    }
}

cudaError_t launch_class_nnz(const LaunchCtx& c, int m) {
    if (m == 0) return cudaSuccess;
    i64 want = ((i64)m + 255) / 256;
    i64 cap = (i64)c.sm_count * 8;
    class_nnz_kernel<<<(int)(want < cap ? want : cap), 256, 0, c.stream>>>(m, c.tab, c.ctl);
    ++c.launches;
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Exclusive scan int32[n] -> int64[n+1] (reduce, scan of block sums, scan): no waits between
// blocks.  out[n] (and *total_out when given) receive the total.
// ---------------------------------------------------------------------------------------
constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = 8;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;

// FLAG: scan (in[i] > 0) instead of in[i] (compaction positions without a flag array).
template <bool FLAG>
__global__ void __launch_bounds__(SCAN_THREADS) scan_reduce_kernel(const int* __restrict__ in, int n, i64* block_sums) {
    __shared__ i64 s_part[SCAN_THREADS / 32];
    const i64 base = (i64)blockIdx.x * SCAN_TILE;
    i64 s = 0;
    for (int x = 0; x < SCAN_ITEMS; ++x) {
        const i64 i = base + x * SCAN_THREADS + threadIdx.x;
        if (i < n) s += FLAG ? (in[i] > 0) : in[i];
    }
    for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        i64 t = 0;
        for (int w = 0; w < SCAN_THREADS / 32; ++w) t += s_part[w];
        block_sums[blockIdx.x] = t;
    }
}

__global__ void __launch_bounds__(1024) scan_block_sums_kernel(i64* block_sums, int nblocks, i64* out_total, i64* total_out2) {
    __shared__ i64 s_warp[32];
    __shared__ i64 s_carry;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    for (int base = 0; base < nblocks; base += 1024) {
        const int i = base + threadIdx.x;
        const i64 v = (i < nblocks) ? block_sums[i] : 0;
        i64 incl = v;
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        for (int d = 1; d < 32; d <<= 1) {
            const i64 t = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += t;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            i64 w = s_warp[lane];
            i64 wi = w;
            for (int d = 1; d < 32; d <<= 1) {
                const i64 t = __shfl_up_sync(0xffffffffu, wi, d);
                if (lane >= d) wi += t;
            }
            s_warp[lane] = wi - w;
        }
        __syncthreads();
        const i64 carry = s_carry;
        if (i < nblocks) block_sums[i] = carry + s_warp[warp] + incl - v;
        __syncthreads();
        if (threadIdx.x == 1023) s_carry = carry + s_warp[warp] + incl;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        *out_total = s_carry;
        if (total_out2) *total_out2 = s_carry;
    }
}

// The in-tile prefix is carried in 64 bits: a tile of 2048 counts may total 2^31 or more.
template <bool FLAG>
__global__ void __launch_bounds__(SCAN_THREADS) scan_apply_kernel(const int* __restrict__ in, int n, const i64* __restrict__ block_sums, i64* __restrict__ out) {
    __shared__ i64 s_warp[SCAN_THREADS / 32];
    const i64 base = (i64)blockIdx.x * SCAN_TILE + (i64)threadIdx.x * SCAN_ITEMS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int v[SCAN_ITEMS];
    i64 s = 0;
#pragma unroll
    for (int x = 0; x < SCAN_ITEMS; ++x) {
        v[x] = (base + x < n) ? (FLAG ? (in[base + x] > 0) : in[base + x]) : 0;
        s += v[x];
    }
    i64 incl = s;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const i64 t = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += t;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    i64 before = 0;
#pragma unroll
    for (int w = 0; w < SCAN_THREADS / 32; ++w) before += (w < warp) ? s_warp[w] : 0;
    i64 run = block_sums[blockIdx.x] + before + incl - s;
#pragma unroll
    for (int x = 0; x < SCAN_ITEMS; ++x) {
        if (base + x < n) out[base + x] = run;
        run += v[x];
    }
}

cudaError_t launch_scan_counts(const LaunchCtx& c, const int* cnt, int n, i64* out, i64* block_sums, i64* total_out, bool as_flags) {
    const int nblocks = (int)(((i64)n + SCAN_TILE - 1) / SCAN_TILE);
    if (nblocks > 0) {
        if (as_flags) scan_reduce_kernel<true><<<nblocks, SCAN_THREADS, 0, c.stream>>>(cnt, n, block_sums);
        else scan_reduce_kernel<false><<<nblocks, SCAN_THREADS, 0, c.stream>>>(cnt, n, block_sums);
    }
    scan_block_sums_kernel<<<1, 1024, 0, c.stream>>>(block_sums, nblocks, out + n, total_out);
    if (nblocks > 0) {
        if (as_flags) scan_apply_kernel<true><<<nblocks, SCAN_THREADS, 0, c.stream>>>(cnt, n, block_sums, out);
        else scan_apply_kernel<false><<<nblocks, SCAN_THREADS, 0, c.stream>>>(cnt, n, block_sums, out);
    }
    c.launches += nblocks > 0 ? 3 : 1;
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// TTM: rebuild C's two upper CSF levels.  A fibre (i,j) survives when it produced at least
// one output; a slice i survives when one of its fibres does.
// ---------------------------------------------------------------------------------------
__global__ void ttm_slice_flags_kernel(int n_i, const i64* __restrict__ Apos1, const i64* __restrict__ fpos, int* sflags) {
    for (i64 s = (i64)blockIdx.x * blockDim.x + threadIdx.x; s < n_i; s += (i64)gridDim.x * blockDim.x)
        sflags[s] = fpos[Apos1[s + 1]] > fpos[Apos1[s]];
}

__global__ void ttm_slice_compact_kernel(int n_i, int n_ij, const int* __restrict__ sflags, const i64* __restrict__ spos,
                                         const i64* __restrict__ Apos1, const i64* __restrict__ fpos,
                                         const int* __restrict__ Acrd0, int* Ccrd0, i64* Cpos1, i64* Cpos0, DevCtl* ctl) {
    for (i64 s = (i64)blockIdx.x * blockDim.x + threadIdx.x; s <= n_i; s += (i64)gridDim.x * blockDim.x) {
        if (s == n_i) {
            Cpos1[spos[n_i]] = fpos[n_ij];
            Cpos0[0] = 0;
            Cpos0[1] = spos[n_i];
            ctl->kept[0] = spos[n_i];
            ctl->kept[1] = fpos[n_ij];
            continue;
        }
        if (sflags[s]) {
            Ccrd0[spos[s]] = Acrd0[s];
            Cpos1[spos[s]] = fpos[Apos1[s]];
        }
    }
}

// The slice level in ONE launch when it is small: a single block flags, scans and compacts the
// slices 1024 at a time with a running count.
__global__ void __launch_bounds__(1024) ttm_slices_small_kernel(int n_i, int n_ij, const i64* __restrict__ Apos1, const i64* __restrict__ fpos,
                                                                const int* __restrict__ Acrd0, int* Ccrd0, i64* Cpos1, i64* Cpos0,
                                                                DevCtl* ctl) {
    __shared__ int ws[33];
    int kept = 0;
    // four consecutive slices per thread, their loads issued together (this block is alone on the
    // GPU, so every dependent load costs a full memory latency)
    for (int s0 = 0; s0 < n_i; s0 += 4096) {
        const int s = s0 + 4 * threadIdx.x;
        i64 edge[5], fp[5];
#pragma unroll
        for (int x = 0; x < 5; ++x) edge[x] = (s + x <= n_i) ? Apos1[s + x] : -1;
#pragma unroll
        for (int x = 0; x < 5; ++x) fp[x] = edge[x] >= 0 ? fpos[edge[x]] : 0;
        int crd[4], nflag = 0;
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const bool flag = s + x < n_i && fp[x + 1] > fp[x];
            crd[x] = flag ? Acrd0[s + x] : -1;
            nflag += flag;
        }
        int total;
        int at = kept + block_excl_scan<1024>(nflag, ws, total);
#pragma unroll
        for (int x = 0; x < 4; ++x)
            if (s + x < n_i && fp[x + 1] > fp[x]) {
                Ccrd0[at] = crd[x];
                Cpos1[at] = fp[x];
                ++at;
            }
        kept += total;
    }
    if (threadIdx.x == 0) {
        Cpos1[kept] = fpos[n_ij];
        Cpos0[0] = 0;
        Cpos0[1] = kept;
        ctl->kept[0] = kept;
        ctl->kept[1] = fpos[n_ij];
    }
}

// The fibre level in three launches: the scan of the counts (C's bottom-level positions) and the
// scan of (count > 0) (where a surviving fibre goes) share their passes over the counts, and the
// second pass places the survivors as it goes.
__global__ void __launch_bounds__(SCAN_THREADS) ttm_dual_reduce_kernel(const int* __restrict__ cnt, int n, i64* sums, i64* kept) {
    __shared__ i64 s_part[2][SCAN_THREADS / 32];
    const i64 base = (i64)blockIdx.x * SCAN_TILE;
    i64 s = 0;
    int k = 0;
    for (int x = 0; x < SCAN_ITEMS; ++x) {
        const i64 i = base + x * SCAN_THREADS + threadIdx.x;
        if (i < n) { const int v = cnt[i]; s += v; k += v > 0; }
    }
    for (int d = 16; d > 0; d >>= 1) {
        s += __shfl_xor_sync(0xffffffffu, s, d);
        k += __shfl_xor_sync(0xffffffffu, k, d);
    }
    if ((threadIdx.x & 31) == 0) { s_part[0][threadIdx.x >> 5] = s; s_part[1][threadIdx.x >> 5] = k; }
    __syncthreads();
    if (threadIdx.x < 2) {
        i64 t = 0;
        for (int w = 0; w < SCAN_THREADS / 32; ++w) t += s_part[threadIdx.x][w];
        (threadIdx.x == 0 ? sums : kept)[blockIdx.x] = t;
    }
}

// exclusive scans of both block-sum arrays by one block; the totals close the three arrays
__global__ void __launch_bounds__(1024) ttm_dual_block_sums_kernel(i64* sums, i64* kept, int nblocks, int n, i64* rowptr_raw, i64* fpos,
                                                                   i64* Cpos2, i64* nnz_out) {
    __shared__ i64 s_warp[2][32];
    __shared__ i64 s_carry[2];
    if (threadIdx.x < 2) s_carry[threadIdx.x] = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int base = 0; base < nblocks; base += 1024) {
        const int i = base + threadIdx.x;
        const i64 v0 = (i < nblocks) ? sums[i] : 0, v1 = (i < nblocks) ? kept[i] : 0;
        i64 i0 = v0, i1 = v1;
        for (int d = 1; d < 32; d <<= 1) {
            const i64 t0 = __shfl_up_sync(0xffffffffu, i0, d), t1 = __shfl_up_sync(0xffffffffu, i1, d);
            if (lane >= d) { i0 += t0; i1 += t1; }
        }
        if (lane == 31) { s_warp[0][warp] = i0; s_warp[1][warp] = i1; }
        __syncthreads();
        if (warp < 2) {
            const i64 w = s_warp[warp][lane];
            i64 wi = w;
            for (int d = 1; d < 32; d <<= 1) {
                const i64 t = __shfl_up_sync(0xffffffffu, wi, d);
                if (lane >= d) wi += t;
            }
            s_warp[warp][lane] = wi - w;
        }
        __syncthreads();
        const i64 c0 = s_carry[0], c1 = s_carry[1];
        if (i < nblocks) { sums[i] = c0 + s_warp[0][warp] + i0 - v0; kept[i] = c1 + s_warp[1][warp] + i1 - v1; }
        __syncthreads();
        if (threadIdx.x == 1023) { s_carry[0] = c0 + s_warp[0][warp] + i0; s_carry[1] = c1 + s_warp[1][warp] + i1; }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        rowptr_raw[n] = s_carry[0];
        fpos[n] = s_carry[1];
        Cpos2[s_carry[1]] = s_carry[0];
        *nnz_out = s_carry[0];
    }
}

__global__ void __launch_bounds__(SCAN_THREADS) ttm_dual_apply_kernel(const int* __restrict__ cnt, int n, const i64* __restrict__ sums,
                                                                      const i64* __restrict__ kept, const int* __restrict__ Acrd1,
                                                                      i64* __restrict__ rowptr_raw, i64* __restrict__ fpos,
                                                                      int* __restrict__ Ccrd1, i64* __restrict__ Cpos2) {
    // a thread scans SCAN_ITEMS consecutive counts; everything crosses shared memory on the way in
    // and out so that global loads and stores are contiguous across the block
    __shared__ i64 s_a[SCAN_TILE];          // counts on the way in (as int), then one output array at a time
    __shared__ int s_crd[SCAN_TILE];        // the tile's fibre coordinates, then the survivors'
    __shared__ i64 s_warp[SCAN_THREADS / 32];
    __shared__ int s_kwarp[SCAN_THREADS / 32];
    const i64 tile = (i64)blockIdx.x * SCAN_TILE;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int len = (int)min((i64)SCAN_TILE, (i64)n - tile);
    int* s_cnt = reinterpret_cast<int*>(s_a);
    for (int i = tid; i < SCAN_TILE; i += SCAN_THREADS) {
        s_cnt[i] = i < len ? cnt[tile + i] : 0;
        s_crd[i] = i < len ? Acrd1[tile + i] : 0;
    }
    __syncthreads();
    int v[SCAN_ITEMS], crd[SCAN_ITEMS];
    i64 s = 0;
    int k = 0;
#pragma unroll
    for (int x = 0; x < SCAN_ITEMS; ++x) {
        v[x] = s_cnt[tid * SCAN_ITEMS + x];
        crd[x] = s_crd[tid * SCAN_ITEMS + x];
        s += v[x];
        k += v[x] > 0;
    }
    i64 incl = s;
    int kincl = k;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const i64 t = __shfl_up_sync(0xffffffffu, incl, d);
        const int tk = __shfl_up_sync(0xffffffffu, kincl, d);
        if (lane >= d) { incl += t; kincl += tk; }
    }
    if (lane == 31) { s_warp[warp] = incl; s_kwarp[warp] = kincl; }
    __syncthreads();                                      // also: every thread has read s_cnt and s_crd
    i64 before = 0;
    int kbefore = 0, ktile = 0;
#pragma unroll
    for (int w = 0; w < SCAN_THREADS / 32; ++w) {
        before += (w < warp) ? s_warp[w] : 0;
        kbefore += (w < warp) ? s_kwarp[w] : 0;
        ktile += s_kwarp[w];
    }
    const i64 run0 = sums[blockIdx.x] + before + incl - s;
    const i64 kept0 = kept[blockIdx.x];
    const int at0 = kbefore + kincl - k;                  // survivors of the tile before this thread's
    // C's bottom-level positions of all fibres
    i64 run = run0;
#pragma unroll
    for (int x = 0; x < SCAN_ITEMS; ++x) { s_a[tid * SCAN_ITEMS + x] = run; run += v[x]; }
    __syncthreads();
    for (int i = tid; i < len; i += SCAN_THREADS) rowptr_raw[tile + i] = s_a[i];
    __syncthreads();
    // place of every fibre among the survivors
    int at = at0;
#pragma unroll
    for (int x = 0; x < SCAN_ITEMS; ++x) { s_a[tid * SCAN_ITEMS + x] = kept0 + at; at += v[x] > 0; }
    __syncthreads();
    for (int i = tid; i < len; i += SCAN_THREADS) fpos[tile + i] = s_a[i];
    __syncthreads();
    // the survivors' coordinates and positions, packed
    run = run0;
    at = at0;
#pragma unroll
    for (int x = 0; x < SCAN_ITEMS; ++x) {
        if (v[x] > 0) { s_a[at] = run; s_crd[at] = crd[x]; ++at; }
        run += v[x];
    }
    __syncthreads();
    for (int i = tid; i < ktile; i += SCAN_THREADS) {
        Cpos2[kept0 + i] = s_a[i];
        Ccrd1[kept0 + i] = s_crd[i];
    }
}

// Scan of the fibre counts, survivors' positions, C's two lower levels' coordinates and positions,
// then the slice level.  `block_sums` holds two arrays of one entry per scan tile.
cudaError_t launch_ttm_scan_compact(const LaunchCtx& c, int n_i, int n_ij, const i64* Apos1, const int* Acrd0, const int* Acrd1,
                                    i64* rowptr_raw, i64* fpos, int* sflags, i64* spos, i64* block_sums, i64* nnz_out,
                                    i64* Cpos0, int* Ccrd0, i64* Cpos1, int* Ccrd1, i64* Cpos2) {
    const int nblocks = (int)(((i64)n_ij + SCAN_TILE - 1) / SCAN_TILE);
    i64* sums = block_sums;
    i64* kept = block_sums + nblocks + 1;
    if (nblocks > 0) ttm_dual_reduce_kernel<<<nblocks, SCAN_THREADS, 0, c.stream>>>(c.tab.cnt, n_ij, sums, kept);
    ttm_dual_block_sums_kernel<<<1, 1024, 0, c.stream>>>(sums, kept, nblocks, n_ij, rowptr_raw, fpos, Cpos2, nnz_out);
    if (nblocks > 0)
        ttm_dual_apply_kernel<<<nblocks, SCAN_THREADS, 0, c.stream>>>(c.tab.cnt, n_ij, sums, kept, Acrd1, rowptr_raw, fpos, Ccrd1, Cpos2);
    c.launches += nblocks > 0 ? 3 : 1;
    if (n_i <= (1 << 16)) {
        ttm_slices_small_kernel<<<1, 1024, 0, c.stream>>>(n_i, n_ij, Apos1, fpos, Acrd0, Ccrd0, Cpos1, Cpos0, c.ctl);
        ++c.launches;
        return cudaGetLastError();
    }
    const int grid = c.sm_count * 8;
    ttm_slice_flags_kernel<<<grid, 256, 0, c.stream>>>(n_i, Apos1, fpos, sflags);
    cudaError_t e = launch_scan_counts(c, sflags, n_i, spos, block_sums, nullptr);
    if (e != cudaSuccess) return e;
    ttm_slice_compact_kernel<<<grid, 256, 0, c.stream>>>(n_i, n_ij, sflags, spos, Apos1, fpos, Acrd0, Ccrd0, Cpos1, Cpos0, c.ctl);
    c.launches += 2;
    return cudaGetLastError();
}

}  // namespace spws

// ---------------------------------------------------------------------------------------
// spws_row_pointer_static: the exclusive scan of the symbolic pass for callers that cannot
// allocate device memory.  The scan's block sums -- the one piece of scratch it needs -- live
// in a fixed array inside the library image instead of a caller-supplied buffer.
// ---------------------------------------------------------------------------------------
#include <mutex>

#include "../../include/spws.h"

namespace {

constexpr long long STATIC_BLOCK_SUMS = SPWS_STATIC_MAX_ROWS / spws::SCAN_TILE;   // 8192 partial sums
static_assert(SPWS_STATIC_MAX_ROWS % spws::SCAN_TILE == 0, "row limit must be a whole number of scan tiles");

// 64 KiB resident on every GPU that loads the library, until the process exits.
static __device__ __align__(256) long long g_static_block_sums[STATIC_BLOCK_SUMS + 2];

constexpr int MAX_DEVICES = 64;
std::mutex g_static_mutex;
void* g_static_addr[MAX_DEVICES] = {};

// The array's name is only a host-side handle; kernels need its device address, which differs
// per GPU and is looked up once per device with that device current.
spws_status_t static_scratch_address(spws::i64** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
        cudaGetLastError();
        return SPWS_CUDA_ERROR;
    }
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_block_sums) != cudaSuccess || !p) {
            cudaGetLastError();
            return SPWS_CUDA_ERROR;
        }
        g_static_addr[dev] = p;
    }
    *out = static_cast<spws::i64*>(g_static_addr[dev]);
    return SPWS_OK;
}

}  // namespace

extern "C" spws_status_t spws_row_pointer_static(const int32_t* counts, int64_t n, int64_t* pos, void* cuda_stream) {
    if (n < 0 || !pos || (n > 0 && !counts)) return SPWS_INVALID_ARGUMENT;
    if (n > SPWS_STATIC_MAX_ROWS) return SPWS_SCRATCH_TOO_SMALL;
    spws::i64* block_sums = nullptr;
    const spws_status_t st = static_scratch_address(&block_sums);
    if (st != SPWS_OK) return st;
    spws::LaunchCtx c{};
    c.stream = static_cast<cudaStream_t>(cuda_stream);
    // Every partial sum the scan reads is written earlier in the same call, so nothing left
    // behind by a previous call has to be cleared.
    if (spws::launch_scan_counts(c, counts, (int)n, reinterpret_cast<spws::i64*>(pos), block_sums, nullptr) != cudaSuccess) {
        cudaGetLastError();
        return SPWS_CUDA_ERROR;
    }
    return SPWS_OK;
}
