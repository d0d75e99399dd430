// Dense workspace in shared memory: a value array plus an occupancy bitmap along the last
// index (Gustavson's workspace, Table 2: a flag marks positions that hold a component, so a
// product deduplicates on insertion; position = coordinate, so the workspace is bucket-sorted;
// the flagged positions are copied out in order = boolean indexing).  A row's column span
// [jmin, jmax] is cut into tiles of W columns; one work unit = (row, tile).  Units of one row
// write disjoint, ordered pieces of the row's output, so hub rows spread over many CTAs
// without atomics between CTAs.
//   symbolic : bitmap only; unit_cnt[u] = popcount; cnt[row] += unit_cnt[u].
//   numeric  : acc[j - c0] += a*b (shared-memory atomics, CTA-wide), then the bitmap is scanned
//              word by word and (j, acc) is written at row_ptr[i] + (outputs of earlier tiles)
//              + rank; touched positions are cleared on the way out.
#include "common.cuh"

namespace spws {

constexpr int DENSE_THREADS = 256;

size_t dense_smem_bytes(int tile_cols, int is_f64) {
    return (size_t)tile_cols * (is_f64 ? 8 : 4) + (size_t)tile_cols / 8 + 16;
}

template <typename T, bool NUMERIC>
__global__ void __launch_bounds__(DENSE_THREADS) dense_unit_kernel(DevCtl* __restrict__ ctl, int counter_slot, int W,
                                                                   Csr A, Csr B, RowTables tab,
                                                                   const i64* __restrict__ rowptr, int* __restrict__ Ccrd, T* __restrict__ Cval) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* acc = reinterpret_cast<T*>(smem_raw);                               // W (numeric only)
    unsigned* bm = reinterpret_cast<unsigned*>(smem_raw + (NUMERIC ? sizeof(T) * (size_t)W : 0));   // W/32
    __shared__ int s_next, s_tile_off;
    __shared__ int ws[33];
    const int tid = threadIdx.x;
    if (ctl->status != 0) return;
    const int n_units = ctl->n_units;
    const T* __restrict__ Aval = (const T*)A.val;
    const T* __restrict__ Bval = (const T*)B.val;

    if (NUMERIC)
        for (int x = tid; x < W; x += DENSE_THREADS) acc[x] = 0;
    for (int x = tid; x < W / 32; x += DENSE_THREADS) bm[x] = 0;

    for (;;) {
        __syncthreads();
        if (tid == 0) s_next = atomicAdd(&ctl->work_counter[counter_slot], 1);
        __syncthreads();
        const int u = s_next;
        if (u >= n_units) break;
        const int row = tab.unit_row[u];
        const int u0 = tab.row_unit0[row];
        const int t = u - u0;
        const int base = tab.jmin[row], last = tab.jmax[row];
        const int ntiles = (last - base) / W + 1;
        const i64 c0 = (i64)base + (i64)t * W;
        const unsigned width = (unsigned)min((i64)W, (i64)last + 1 - c0);
        const i64 ps = A.pos[row], pe = A.pos[row + 1];

        if (NUMERIC && tid < 32) {          // outputs of the earlier tiles of this row
            int s = 0;
            for (int x = tid; x < t; x += 32) s += tab.unit_cnt[u0 + x];
            for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
            if (tid == 0) s_tile_off = s;
        }

        // lanes per A entry: about the expected length of a B-row segment inside this tile
        int gs = 32;
        {
            const i64 nA = pe - ps;
            const i64 avg = tab.ub[row] / (nA * ntiles > 0 ? nA * ntiles : 1);
            while (gs > 1 && (gs >> 1) >= avg) gs >>= 1;
        }
        const int g = tid / gs, gl = tid % gs, ngroups = DENSE_THREADS / gs;
        for (i64 p = ps + g; p < pe; p += ngroups) {
            const int k = __ldg(A.crd + p);
            if ((unsigned)k >= (unsigned)B.nrows) continue;
            i64 qs = __ldg(B.pos + k);
            const i64 qe = __ldg(B.pos + k + 1);
            if (ntiles > 1) qs = lower_bound_crd(B.crd, qs, qe, (int)c0);
            T a = 0;
            if (NUMERIC) a = __ldg(Aval + p);
            for (i64 q = qs + gl; q < qe; q += gs) {
                const unsigned rel = (unsigned)((i64)__ldg(B.crd + q) - c0);
                if (rel >= width) break;
                if (NUMERIC) atomicAdd(&acc[rel], a * __ldg(Bval + q));
                atomicOr(&bm[rel >> 5], 1u << (rel & 31));
            }
        }
        __syncthreads();

        // ---- copy out in coordinate order
        const int nwords = (int)((width + 31) >> 5);
        int running = 0;
        const i64 out0 = NUMERIC ? rowptr[row] + s_tile_off : 0;
        for (int w0 = 0; w0 < nwords; w0 += DENSE_THREADS) {
            const int w = w0 + tid;
            unsigned bits = (w < nwords) ? bm[w] : 0u;
            int chunk_total;
            const int off = block_excl_scan<DENSE_THREADS>(__popc(bits), ws, chunk_total);
            if (bits) {
                bm[w] = 0;
                if (NUMERIC) {
                    i64 out = out0 + running + off;
                    while (bits) {
                        const int b = __ffs(bits) - 1;
                        bits &= bits - 1;
                        const int rel = (w << 5) + b;
                        Ccrd[out] = (int)(c0 + rel);
                        Cval[out] = acc[rel];
                        acc[rel] = 0;
                        ++out;
                    }
                }
            }
            running += chunk_total;
        }
        if (!NUMERIC && tid == 0) {
            tab.unit_cnt[u] = running;
            atomicAdd(&tab.cnt[row], running);
        }
    }
}

template <typename T>
static cudaError_t launch_t(const LaunchCtx& c, bool numeric, int n_units_host, const Csr& A, const Csr& B,
                            const i64* rowptr, int* Ccrd, void* Cval) {
    const int W = c.prm.tile_cols;
    const size_t smem = (numeric ? sizeof(T) * (size_t)W : 0) + (size_t)W / 8 + 16;
    const int slot = CLS_DENSE + (numeric ? 8 : 0);
    cudaError_t e;
    int per_sm = 0;
    if (numeric) {
        auto k = dense_unit_kernel<T, true>;
        if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, DENSE_THREADS, smem)) != cudaSuccess) return e;
        i64 grid = (i64)c.sm_count * (per_sm > 0 ? per_sm : 1);
        if (n_units_host >= 0 && n_units_host < grid) grid = n_units_host > 0 ? n_units_host : 1;
        k<<<(int)grid, DENSE_THREADS, smem, c.stream>>>(c.ctl, slot, W, A, B, c.tab, rowptr, Ccrd, (T*)Cval);
    } else {
        auto k = dense_unit_kernel<T, false>;
        if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, DENSE_THREADS, smem)) != cudaSuccess) return e;
        i64 grid = (i64)c.sm_count * (per_sm > 0 ? per_sm : 1);
        if (n_units_host >= 0 && n_units_host < grid) grid = n_units_host > 0 ? n_units_host : 1;
        k<<<(int)grid, DENSE_THREADS, smem, c.stream>>>(c.ctl, slot, W, A, B, c.tab, rowptr, Ccrd, (T*)Cval);
    }
    ++c.launches;
    return cudaGetLastError();
}

cudaError_t launch_dense(const LaunchCtx& c, bool numeric, int n_units_host, const Csr& A, const Csr& B,
                         const i64* rowptr, int* Ccrd, void* Cval) {
    return c.is_f64 ? launch_t<double>(c, numeric, n_units_host, A, B, rowptr, Ccrd, Cval)
                    : launch_t<float>(c, numeric, n_units_host, A, B, rowptr, Ccrd, Cval);
}

}  // namespace spws
