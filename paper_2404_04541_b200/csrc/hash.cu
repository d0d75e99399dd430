// Hash workspace: insert-sort-merge with the reduction done at insert time (Sec. 4.3 allows
// duplicates to be reduced "during the insertion stage"; Sec. 5.2's Bucket / Hash policies keep a
// table so that an insertion finds an equal coordinate at once; Table 2's hash-based SpGEMM row).
// One CTA per output row whose product count is at most CAP:
//   Insert : product t of the row looks its column up in an open-addressing table in shared memory
//            (multiplicative hash, linear probing; the table has at least twice as many slots as
//            the row can have distinct columns, so it never fills).  A new column claims a slot
//            with a compare-and-swap on the key; the value is added to the slot.
//   Sort   : only the DISTINCT columns are sorted -- the occupied slots are compacted into
//            (column, slot) words and put in order by a bitonic network.
//   Merge  : nothing is left to reduce; the sorted words are written out with their slots' sums.
// The symbolic pass runs the same insertions on keys only and counts the claims.
#include "common.cuh"

namespace spws {

constexpr int HASH_EMPTY = -1;

template <typename T, int CAP, int THREADS, bool NUMERIC>
__global__ void __launch_bounds__(THREADS) hash_kernel(const int* __restrict__ perm, DevCtl* __restrict__ ctl, int cls, int counter_slot,
                                                       Csr A, Csr B, const i64* __restrict__ ub, int* __restrict__ cnt,
                                                       const i64* __restrict__ rowptr, int* __restrict__ Ccrd, T* __restrict__ Cval) {
    constexpr int SLOTS = 2 * CAP;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* vals = reinterpret_cast<T*>(smem_raw);                             // SLOTS (numeric only)
    int* keys = reinterpret_cast<int*>(vals + (NUMERIC ? SLOTS : 0));     // SLOTS
    u64* packed = reinterpret_cast<u64*>(keys + SLOTS);                   // CAP (numeric only)
    i64* e_qs = reinterpret_cast<i64*>(packed + (NUMERIC ? CAP : 0));     // THREADS
    T* e_a = reinterpret_cast<T*>(e_qs + THREADS);                        // THREADS
    int* e_off = reinterpret_cast<int*>(e_a + THREADS);                   // THREADS + 1
    int* ws = e_off + THREADS + 1;                                        // 33
    __shared__ int s_next, s_n;

    if (ctl->status != 0) return;
    int off, n;
    class_range(ctl, cls, off, n);
    const int* __restrict__ rows = perm + off;
    const T* __restrict__ Aval = (const T*)A.val;
    const T* __restrict__ Bval = (const T*)B.val;
    const int tid = threadIdx.x;

    for (;;) {
        __syncthreads();
        if (tid == 0) { s_next = atomicAdd(&ctl->work_counter[counter_slot], 1); s_n = 0; }
        __syncthreads();
        const int r = s_next;
        if (r >= n) break;
        const int row = rows[r];
        const i64 ps = A.pos[row], pe = A.pos[row + 1];
        // the numeric pass knows the row's distinct columns and sizes the table from them
        // (the counting pass sizes it from the row's product count, an upper bound of them)
        int slots = 16;
        i64 out0 = 0;
        int row_cnt = 0;
        if (NUMERIC) {
            out0 = rowptr[row];
            row_cnt = min((int)(rowptr[row + 1] - out0), CAP);
            while (slots < 2 * row_cnt) slots <<= 1;
        } else {
            const int bound = (int)min(ub[row], (i64)CAP);
            while (slots < 2 * bound) slots <<= 1;
        }
        const unsigned mask = (unsigned)slots - 1u;
        const int shift = 32 - __popc(mask);
        for (int x = tid; x < slots; x += THREADS) {
            keys[x] = HASH_EMPTY;
            if (NUMERIC) vals[x] = 0;
        }
        __syncthreads();

        // ---- Insert (reduces on the spot)
        int claims = 0;
        for (i64 p0 = ps; p0 < pe; p0 += THREADS) {
            const i64 p = p0 + tid;
            int len = 0;
            i64 qs = 0;
            T a = 0;
            if (p < pe) {
                const int k = __ldg(A.crd + p);
                if ((unsigned)k < (unsigned)B.nrows) {
                    qs = __ldg(B.pos + k);
                    len = (int)(__ldg(B.pos + k + 1) - qs);
                }
                if (NUMERIC) a = __ldg(Aval + p);
            }
            int chunk_total;
            const int excl = block_excl_scan<THREADS>(len, ws, chunk_total);
            e_off[tid] = excl;
            e_qs[tid] = qs;
            if (NUMERIC) e_a[tid] = a;
            if (tid == 0) e_off[THREADS] = chunk_total;
            __syncthreads();
            const int nE = (int)min((i64)THREADS, pe - p0);
            for (int t = tid; t < chunk_total; t += THREADS) {
                int lo = 0, hi = nE;
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (e_off[mid] <= t) lo = mid; else hi = mid;
                }
                const i64 q = e_qs[lo] + (t - e_off[lo]);
                const int col = __ldg(B.crd + q);
                unsigned h = ((unsigned)col * 2654435761u) >> shift;
                int probes = 0;
                for (;; ++probes) {
                    if (probes >= slots) { raise_status(ctl, DEV_INTERNAL_OVERFLOW); break; }
                    const int seen = ((volatile int*)keys)[h];
                    if (seen == col) break;
                    if (seen == HASH_EMPTY) {
                        const int old = atomicCAS(&keys[h], HASH_EMPTY, col);
                        if (old == HASH_EMPTY) { ++claims; break; }
                        if (old == col) break;
                    }
                    h = (h + 1u) & mask;
                }
                if (NUMERIC && probes < slots) atomicAdd(&vals[h], mul_rn(e_a[lo], __ldg(Bval + q)));
            }
            __syncthreads();
        }
        if (!NUMERIC) {
            int total;
            block_excl_scan<THREADS>(claims, ws, total);
            if (tid == 0) cnt[row] = total;
            continue;
        }

        // ---- Sort the distinct columns: compact (column, slot), bitonic network
        for (int x = tid; x < slots; x += THREADS) {
            const int key = keys[x];
            if (key != HASH_EMPTY) {
                const int at = atomicAdd(&s_n, 1);
                if (at < CAP) packed[at] = ((u64)(unsigned)key << 32) | (unsigned)x;
            }
        }
        __syncthreads();
        const int total = min(s_n, CAP);
        int n2 = 1;
        while (n2 < total) n2 <<= 1;
        for (int t = total + tid; t < n2; t += THREADS) packed[t] = ~0ull;
        __syncthreads();
        for (int k = 2; k <= n2; k <<= 1) {
            for (int j = k >> 1; j > 0; j >>= 1) {
                for (int t = tid; t < (n2 >> 1); t += THREADS) {
                    const int i = 2 * t - (t & (j - 1));
                    const int l = i + j;
                    const u64 x = packed[i], y = packed[l];
                    const bool up = (i & k) == 0;
                    if ((x > y) == up) { packed[i] = y; packed[l] = x; }
                }
                __syncthreads();
            }
        }
        // ---- write out (Merge has nothing left to do)
        for (int x = tid; x < min(total, row_cnt); x += THREADS) {
            const u64 w = packed[x];
            Ccrd[out0 + x] = (int)(unsigned)(w >> 32);
            Cval[out0 + x] = vals[(unsigned)w];
        }
    }
}

template <typename T, int CAP, int THREADS>
static size_t hash_smem_bytes(bool numeric) {
    const size_t slots = 2 * (size_t)CAP;
    return (numeric ? sizeof(T) * slots : 0) + 4 * slots + (numeric ? 8 * (size_t)CAP : 0) + sizeof(i64) * THREADS + sizeof(T) * THREADS +
           sizeof(int) * (THREADS + 1 + 33) + 16;
}

template <typename T, int CAP, int THREADS, bool NUMERIC>
static cudaError_t hash_launch_k(const LaunchCtx& c, int cls, int n_host, const Csr& A, const Csr& B, const i64* rowptr, int* Ccrd, void* Cval) {
    const size_t smem = hash_smem_bytes<T, CAP, THREADS>(NUMERIC);
    const int slot = cls + (NUMERIC ? NUM_SLOT : 0);
    cudaError_t e;
    int per_sm = 0;
    auto k = hash_kernel<T, CAP, THREADS, NUMERIC>;
    if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, THREADS, smem)) != cudaSuccess) return e;
    i64 grid = (i64)c.sm_count * (per_sm > 0 ? per_sm : 1);
    if (n_host >= 0 && n_host < grid) grid = n_host > 0 ? n_host : 1;
    k<<<(int)grid, THREADS, smem, c.stream>>>(c.tab.perm, c.ctl, cls, slot, A, B, c.tab.ub, c.tab.cnt, rowptr, Ccrd, (T*)Cval);
    ++c.launches;
    return cudaGetLastError();
}

template <typename T>
static cudaError_t hash_launch_t(const LaunchCtx& c, bool numeric, int cls, int n_host, const Csr& A, const Csr& B, const i64* rowptr,
                                 int* Ccrd, void* Cval) {
    // the counting pass also serves the shared-memory insert-sort-merge classes (no sort is needed to
    // count distinct columns); their rows have at most HASH_CAP products
    if (!numeric && cls == CLS_ISM_SMEM_S) return hash_launch_k<T, HASH_SMALL_CAP, 128, false>(c, cls, n_host, A, B, rowptr, Ccrd, Cval);
    if (!numeric && cls == CLS_ISM_SMEM) return hash_launch_k<T, HASH_CAP, 256, false>(c, cls, n_host, A, B, rowptr, Ccrd, Cval);
    if (cls == CLS_HASH_S)
        return numeric ? hash_launch_k<T, HASH_SMALL_CAP, 128, true>(c, cls, n_host, A, B, rowptr, Ccrd, Cval)
                       : hash_launch_k<T, HASH_SMALL_CAP, 128, false>(c, cls, n_host, A, B, rowptr, Ccrd, Cval);
    return numeric ? hash_launch_k<T, HASH_CAP, 256, true>(c, cls, n_host, A, B, rowptr, Ccrd, Cval)
                   : hash_launch_k<T, HASH_CAP, 256, false>(c, cls, n_host, A, B, rowptr, Ccrd, Cval);
}

cudaError_t launch_hash(const LaunchCtx& c, bool numeric, int cls, int n_host, const Csr& A, const Csr& B, const i64* rowptr,
                        int* Ccrd, void* Cval) {
    return c.is_f64 ? hash_launch_t<double>(c, numeric, cls, n_host, A, B, rowptr, Ccrd, Cval)
                    : hash_launch_t<float>(c, numeric, cls, n_host, A, B, rowptr, Ccrd, Cval);
}

}  // namespace spws
