// Insert-sort-merge with the all array in global memory, for rows whose products overflow
// shared memory (Algorithm 1 taken whole; coordinate-sort policy, Sec. 5.2).
//   Allocate : the accumulation array (capacity `cap` components) lives in shared memory; the
//              all array is a pair of buffers in the caller's scratch, one slot per CTA
//              (double buffering, Sec. 5.3: Merge is out of place, the buffers swap roles).
//   Insert   : the next `cap` products of the row, in loop order, are appended; the array is
//              full exactly when `cap` products are in, and the product that did not fit opens
//              the next round (the Insert / full / Insert-again protocol of Algorithm 1).
//   Sort     : bitonic sort on (j << 32 | slot); equal coordinates are reduced in slot order.
//   Merge    : two-way merge of the sorted, unique accumulation array with the sorted, unique
//              all array, equal coordinates reduced.  Each side finds its output position by
//              binary search in the other (the data-parallel form of the O(n+m) merge).
//   Compress : the all array is copied to the row's segment of C (numeric) or its length is
//              the row's output count (symbolic).
#include "common.cuh"

namespace spws {

constexpr int GL_THREADS = 256;
constexpr int GL_CAPMAX = 2048;

template <typename T, bool NUMERIC>
__global__ void __launch_bounds__(GL_THREADS) ism_global_kernel(const int* __restrict__ perm, DevCtl* __restrict__ ctl, int counter_slot,
                                                                int cap, char* rest, size_t rest_bytes,
                                                                Csr A, Csr B, int* __restrict__ cnt,
                                                                const i64* __restrict__ rowptr, int* __restrict__ Ccrd, T* __restrict__ Cval) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    u64* packed = reinterpret_cast<u64*>(smem_raw);                  // GL_CAPMAX
    T* vals = reinterpret_cast<T*>(packed + GL_CAPMAX);              // GL_CAPMAX
    T* uvals = vals + GL_CAPMAX;                                     // GL_CAPMAX
    i64* e_qs = reinterpret_cast<i64*>(uvals + GL_CAPMAX);           // GL_THREADS
    T* e_a = reinterpret_cast<T*>(e_qs + GL_THREADS);                // GL_THREADS
    int* ukeys = reinterpret_cast<int*>(e_a + GL_THREADS);           // GL_CAPMAX
    int* upos = ukeys + GL_CAPMAX;                                   // GL_CAPMAX
    int* unew = upos + GL_CAPMAX;                                    // GL_CAPMAX + 1 : unmatched prefix
    int* e_off = unew + GL_CAPMAX + 1;                               // GL_THREADS + 1
    int* ws = e_off + GL_THREADS + 1;                                // 33
    __shared__ int s_next;

    if (ctl->status != 0) return;
    int off, n;
    class_range(ctl, CLS_ISM_GLOBAL, off, n);
    if (n == 0) return;
    const int* __restrict__ rows = perm + off;
    const T* __restrict__ Aval = (const T*)A.val;
    const T* __restrict__ Bval = (const T*)B.val;
    const int tid = threadIdx.x;

    // the arena follows the bitmap arena in the rest of the scratch buffer
    const size_t bm_bytes = ((size_t)ctl->bm_words_used * 4 + 255) & ~(size_t)255;
    char* arena = rest + bm_bytes;
    const size_t arena_bytes = rest_bytes > bm_bytes ? rest_bytes - bm_bytes : 0;
    // one slot per CTA: two all-array buffers of slot_elems components
    i64 slot_elems = min(ctl->max_ub_global, (i64)B.ncols);
    slot_elems = (slot_elems + 63) & ~63ll;
    const size_t comp_bytes = sizeof(int) + (NUMERIC ? sizeof(T) : 0);
    const size_t slot_bytes = (2 * (size_t)slot_elems * comp_bytes + 255) & ~(size_t)255;
    const i64 nslots = (i64)(arena_bytes / slot_bytes);
    if (nslots == 0) {
        if (blockIdx.x == 0 && tid == 0) raise_status(ctl, DEV_SCRATCH_TOO_SMALL);
        return;
    }
    if (blockIdx.x >= nslots) return;
    char* slot = arena + (size_t)blockIdx.x * slot_bytes;
    int* all_key[2] = {reinterpret_cast<int*>(slot), reinterpret_cast<int*>(slot) + slot_elems};
    T* all_val[2] = {reinterpret_cast<T*>(slot + 2 * (size_t)slot_elems * sizeof(int)),
                     reinterpret_cast<T*>(slot + 2 * (size_t)slot_elems * sizeof(int)) + slot_elems};

    for (;;) {
        __syncthreads();
        if (tid == 0) s_next = atomicAdd(&ctl->work_counter[counter_slot], 1);
        __syncthreads();
        const int r = s_next;
        if (r >= n) break;
        const int row = rows[r];
        const i64 ps = A.pos[row], pe = A.pos[row + 1];

        int all_n = 0, cur = 0;
        i64 p_cur = ps;       // next A entry of the product stream
        int q_skip = 0;       // products of entry p_cur already consumed
        while (p_cur < pe) {
            // ---- Insert: up to `cap` products
            int acc_n = 0;
            while (p_cur < pe && acc_n < cap) {
                const i64 p = p_cur + tid;
                int len = 0;
                i64 qs = 0;
                T a = 0;
                if (p < pe) {
                    const int k = __ldg(A.crd + p);
                    if ((unsigned)k < (unsigned)B.nrows) {
                        qs = __ldg(B.pos + k);
                        len = (int)(__ldg(B.pos + k + 1) - qs);
                    }
                    if (tid == 0) { qs += q_skip; len -= q_skip; }
                    if (NUMERIC) a = __ldg(Aval + p);
                }
                int chunk_total;
                const int excl = block_excl_scan<GL_THREADS>(len, ws, chunk_total);
                e_off[tid] = excl;
                e_qs[tid] = qs;
                if (NUMERIC) e_a[tid] = a;
                if (tid == 0) e_off[GL_THREADS] = chunk_total;
                __syncthreads();
                const int nE = (int)min((i64)GL_THREADS, pe - p_cur);
                const int take = min(chunk_total, cap - acc_n);
                for (int t = tid; t < take; t += GL_THREADS) {
                    int lo = 0, hi = nE;
                    while (hi - lo > 1) {
                        const int mid = (lo + hi) >> 1;
                        if (e_off[mid] <= t) lo = mid; else hi = mid;
                    }
                    const i64 q = e_qs[lo] + (t - e_off[lo]);
                    const int s = acc_n + t;
                    packed[s] = ((u64)(unsigned)__ldg(B.crd + q) << 32) | (unsigned)s;
                    if (NUMERIC) vals[s] = mul_rn(e_a[lo], __ldg(Bval + q));
                }
                if (take < chunk_total) {
                    // the array is full: product number `take` of this chunk is the one that did
                    // not fit; it opens the next round
                    int lo = 0, hi = nE;
                    while (hi - lo > 1) {
                        const int mid = (lo + hi) >> 1;
                        if (e_off[mid] <= take) lo = mid; else hi = mid;
                    }
                    const int within = take - e_off[lo];
                    q_skip = (lo == 0 ? q_skip : 0) + within;
                    p_cur += lo;
                } else {
                    p_cur += nE;
                    q_skip = 0;
                }
                acc_n += take;
                __syncthreads();
            }
            if (acc_n == 0) break;

            // ---- Sort
            int n2 = 1;
            while (n2 < acc_n) n2 <<= 1;
            for (int t = acc_n + tid; t < n2; t += GL_THREADS) packed[t] = ~0ull;
            __syncthreads();
            for (int k = 2; k <= n2; k <<= 1) {
                for (int j = k >> 1; j > 0; j >>= 1) {
                    for (int t = tid; t < (n2 >> 1); t += GL_THREADS) {
                        const int i = 2 * t - (t & (j - 1));
                        const int l = i + j;
                        const u64 x = packed[i], y = packed[l];
                        const bool up = (i & k) == 0;
                        if ((x > y) == up) { packed[i] = y; packed[l] = x; }
                    }
                    __syncthreads();
                }
            }
            // reduce equal coordinates -> ukeys/uvals[0, m)
            const int chunk = (acc_n + GL_THREADS - 1) / GL_THREADS;
            const int x0 = min(acc_n, tid * chunk), x1 = min(acc_n, x0 + chunk);
            int heads = 0;
            for (int x = x0; x < x1; ++x)
                heads += (x == 0) || ((unsigned)(packed[x] >> 32) != (unsigned)(packed[x - 1] >> 32));
            int m;
            int rank = block_excl_scan<GL_THREADS>(heads, ws, m);
            for (int x = x0; x < x1; ++x) {
                const unsigned key = (unsigned)(packed[x] >> 32);
                if (x != 0 && key == (unsigned)(packed[x - 1] >> 32)) continue;
                if (NUMERIC) {
                    T sum = vals[(unsigned)packed[x]];
                    for (int y = x + 1; y < acc_n && (unsigned)(packed[y] >> 32) == key; ++y)
                        sum = add_rn(sum, vals[(unsigned)packed[y]]);
                    uvals[rank] = sum;
                }
                ukeys[rank] = (int)key;
                ++rank;
            }
            __syncthreads();

            // ---- Merge(Acc, All): positions by mutual binary search
            // plain pointers: these buffers are written and re-read inside this kernel
            const int* ak = all_key[cur];
            const T* av = all_val[cur];
            int* ok = all_key[cur ^ 1];
            T* ov = all_val[cur ^ 1];
            const int mchunk = (m + GL_THREADS - 1) / GL_THREADS;
            const int m0 = min(m, tid * mchunk), m1 = min(m, m0 + mchunk);
            int fresh = 0;
            for (int x = m0; x < m1; ++x) {
                const int key = ukeys[x];
                int lo = 0, hi = all_n;
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (ak[mid] < key) lo = mid + 1; else hi = mid;
                }
                const bool match = lo < all_n && ak[lo] == key;
                upos[x] = match ? -1 : lo;
                fresh += !match;
            }
            int n_fresh;
            int frank = block_excl_scan<GL_THREADS>(fresh, ws, n_fresh);
            if (all_n + n_fresh > slot_elems) {          // cannot happen: uniques <= min(ub, ncols)
                if (tid == 0) raise_status(ctl, DEV_INTERNAL_OVERFLOW);
                all_n = 0;
                break;
            }
            for (int x = m0; x < m1; ++x) {
                unew[x] = frank;
                if (upos[x] >= 0) {
                    const int o = upos[x] + frank;
                    ok[o] = ukeys[x];
                    if (NUMERIC) ov[o] = uvals[x];
                    ++frank;
                }
            }
            if (tid == 0) unew[m] = n_fresh;
            __syncthreads();
            for (int y = tid; y < all_n; y += GL_THREADS) {
                const int key = ak[y];
                int lo = 0, hi = m;
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (ukeys[mid] < key) lo = mid + 1; else hi = mid;
                }
                const int o = y + unew[lo];
                ok[o] = key;
                if (NUMERIC) ov[o] = (lo < m && ukeys[lo] == key) ? add_rn(av[y], uvals[lo]) : av[y];
            }
            all_n += n_fresh;
            cur ^= 1;
            __syncthreads();
        }

        // ---- Compress
        if (!NUMERIC) {
            if (tid == 0) cnt[row] = all_n;
        } else {
            const i64 out0 = rowptr[row];
            for (int y = tid; y < all_n; y += GL_THREADS) {
                Ccrd[out0 + y] = all_key[cur][y];
                Cval[out0 + y] = all_val[cur][y];
            }
        }
    }
}

template <typename T>
static cudaError_t launch_t(const LaunchCtx& c, bool numeric, int n_host, const Csr& A, const Csr& B,
                            const i64* rowptr, int* Ccrd, void* Cval) {
    const size_t smem = sizeof(u64) * GL_CAPMAX + sizeof(T) * GL_CAPMAX * 2 + sizeof(i64) * GL_THREADS + sizeof(T) * GL_THREADS +
                        sizeof(int) * (3 * GL_CAPMAX + 1 + GL_THREADS + 1 + 33) + 16;
    const int slot = CLS_ISM_GLOBAL + (numeric ? NUM_SLOT : 0);
    cudaError_t e;
    i64 grid = (i64)c.sm_count * 2;
    if (n_host >= 0 && n_host < grid) grid = n_host > 0 ? n_host : 1;
    if (numeric) {
        auto k = ism_global_kernel<T, true>;
        if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        k<<<(int)grid, GL_THREADS, smem, c.stream>>>(c.tab.perm, c.ctl, slot, c.global_cap, c.rest, c.rest_bytes,
                                                    A, B, c.tab.cnt, rowptr, Ccrd, (T*)Cval);
    } else {
        auto k = ism_global_kernel<T, false>;
        if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        k<<<(int)grid, GL_THREADS, smem, c.stream>>>(c.tab.perm, c.ctl, slot, c.global_cap, c.rest, c.rest_bytes,
                                                    A, B, c.tab.cnt, rowptr, Ccrd, (T*)Cval);
    }
    ++c.launches;
    return cudaGetLastError();
}

cudaError_t launch_ism_global(const LaunchCtx& c, bool numeric, int n_host, const Csr& A, const Csr& B,
                              const i64* rowptr, int* Ccrd, void* Cval) {
    return c.is_f64 ? launch_t<double>(c, numeric, n_host, A, B, rowptr, Ccrd, Cval)
                    : launch_t<float>(c, numeric, n_host, A, B, rowptr, Ccrd, Cval);
}

}  // namespace spws
