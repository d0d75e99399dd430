// Insert-sort-merge workspace in shared memory: one CTA per output row with at most CAP
// products (Algorithm 1; the accumulation array is the CTA's shared memory and is never full
// because the symbolic upper bound sized it; coordinate-sort policy, Sec. 5.2).
//   Insert : product t of the row (loop order k, then j) is appended at slot t: its value stays
//            there, and the packed word (j, t) enters the sort (accumulation indexing, Sec. 5.1:
//            only integers move).  The word is 32 bits (j << log2 CAP | t) when the column count
//            leaves room for it, else 64 bits (j << 32 | t).
//   Sort   : bitonic sort of the packed words (lexicographic on (j, t), hence stable).
//   Merge  : runs of equal j are reduced in slot order and written at row_ptr[i] + rank.
#include "common.cuh"

namespace spws {

template <int CAP> struct Log2 { static constexpr int value = 1 + Log2<CAP / 2>::value; };
template <> struct Log2<1> { static constexpr int value = 0; };

// packed (column, slot) words
template <typename P, int CAP> struct Pack;
template <int CAP> struct Pack<u64, CAP> {
    static __device__ __forceinline__ u64 make(int col, int slot) { return ((u64)(unsigned)col << 32) | (unsigned)slot; }
    static __device__ __forceinline__ unsigned key(u64 p) { return (unsigned)(p >> 32); }
    static __device__ __forceinline__ unsigned slot(u64 p) { return (unsigned)p; }
    static __device__ __forceinline__ u64 sentinel() { return ~0ull; }
};
template <int CAP> struct Pack<unsigned, CAP> {
    static constexpr int LG = Log2<CAP>::value;
    static __device__ __forceinline__ unsigned make(int col, int slot) { return ((unsigned)col << LG) | (unsigned)slot; }
    static __device__ __forceinline__ unsigned key(unsigned p) { return p >> LG; }
    static __device__ __forceinline__ unsigned slot(unsigned p) { return p & (unsigned)(CAP - 1); }
    static __device__ __forceinline__ unsigned sentinel() { return ~0u; }
};

template <typename T, typename P, int CAP, int THREADS, bool NUMERIC>
__global__ void __launch_bounds__(THREADS) ism_smem_kernel(const int* __restrict__ perm, DevCtl* __restrict__ ctl, int cls,
                                                           int counter_slot, Csr A, Csr B, int* __restrict__ cnt,
                                                           const i64* __restrict__ rowptr, int* __restrict__ Ccrd, T* __restrict__ Cval) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    typedef Pack<P, CAP> PK;
    T* vals = reinterpret_cast<T*>(smem_raw);                             // CAP (numeric only)
    P* packed = reinterpret_cast<P*>(vals + (NUMERIC ? CAP : 0));         // CAP
    i64* e_qs = reinterpret_cast<i64*>(smem_raw + (((NUMERIC ? sizeof(T) * CAP : 0) + sizeof(P) * CAP + 7) & ~(size_t)7));   // THREADS
    T* e_a = reinterpret_cast<T*>(e_qs + THREADS);                        // THREADS
    int* e_off = reinterpret_cast<int*>(e_a + THREADS);                   // THREADS + 1
    int* ws = e_off + THREADS + 1;                                        // 33
    __shared__ int s_next;

    if (ctl->status != 0) return;
    int off, n;
    class_range(ctl, cls, off, n);
    const int* __restrict__ rows = perm + off;
    const T* __restrict__ Aval = (const T*)A.val;
    const T* __restrict__ Bval = (const T*)B.val;
    const int tid = threadIdx.x;

    for (;;) {
        __syncthreads();
        if (tid == 0) s_next = atomicAdd(&ctl->work_counter[counter_slot], 1);
        __syncthreads();
        const int r = s_next;
        if (r >= n) break;
        const int row = rows[r];
        const i64 ps = A.pos[row], pe = A.pos[row + 1];

        // ---- Insert
        int total = 0;
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
            if (total + chunk_total > CAP) chunk_total = CAP - total;     // cannot happen for a correctly classed row
            for (int t = tid; t < chunk_total; t += THREADS) {
                int lo = 0, hi = nE;
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (e_off[mid] <= t) lo = mid; else hi = mid;
                }
                const i64 q = e_qs[lo] + (t - e_off[lo]);
                const int slot = total + t;
                packed[slot] = PK::make(__ldg(B.crd + q), slot);
                if (NUMERIC) vals[slot] = mul_rn(e_a[lo], __ldg(Bval + q));
            }
            total += chunk_total;
            __syncthreads();
        }
        int n2 = 1;
        while (n2 < total) n2 <<= 1;
        for (int t = total + tid; t < n2; t += THREADS) packed[t] = PK::sentinel();
        __syncthreads();

        // ---- Sort
        for (int k = 2; k <= n2; k <<= 1) {
            for (int j = k >> 1; j > 0; j >>= 1) {
                for (int t = tid; t < (n2 >> 1); t += THREADS) {
                    const int i = 2 * t - (t & (j - 1));
                    const int l = i + j;
                    const P x = packed[i], y = packed[l];
                    const bool up = (i & k) == 0;
                    if ((x > y) == up) { packed[i] = y; packed[l] = x; }
                }
                __syncthreads();
            }
        }

        // ---- Merge
        const int chunk = (total + THREADS - 1) / THREADS;
        const int x0 = min(total, tid * chunk), x1 = min(total, x0 + chunk);
        int heads = 0;
        for (int x = x0; x < x1; ++x)
            heads += (x == 0) || (PK::key(packed[x]) != PK::key(packed[x - 1]));
        int row_cnt;
        int rank = block_excl_scan<THREADS>(heads, ws, row_cnt);
        if (!NUMERIC) {
            if (tid == 0) cnt[row] = row_cnt;
        } else {
            const i64 out0 = rowptr[row];
            for (int x = x0; x < x1; ++x) {
                const unsigned key = PK::key(packed[x]);
                if (x != 0 && key == PK::key(packed[x - 1])) continue;
                T sum = vals[PK::slot(packed[x])];
                for (int y = x + 1; y < total && PK::key(packed[y]) == key; ++y)
                    sum = add_rn(sum, vals[PK::slot(packed[y])]);
                Ccrd[out0 + rank] = (int)key;
                Cval[out0 + rank] = sum;
                ++rank;
            }
        }
    }
}

template <typename T, typename P, int CAP, int THREADS>
static size_t smem_bytes(bool numeric) {
    return (((numeric ? sizeof(T) * CAP : 0) + sizeof(P) * CAP + 7) & ~(size_t)7) + sizeof(i64) * THREADS + sizeof(T) * THREADS +
           sizeof(int) * (THREADS + 1 + 33) + 16;
}

template <typename T, typename P, int CAP, int THREADS, bool NUMERIC>
static cudaError_t launch_k(const LaunchCtx& c, int cls, int n_host, const Csr& A, const Csr& B,
                            const i64* rowptr, int* Ccrd, void* Cval) {
    const size_t smem = smem_bytes<T, P, CAP, THREADS>(NUMERIC);
    const int slot = cls + (NUMERIC ? NUM_SLOT : 0);
    cudaError_t e;
    int per_sm = 0;
    auto k = ism_smem_kernel<T, P, CAP, THREADS, NUMERIC>;
    if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, THREADS, smem)) != cudaSuccess) return e;
    i64 grid = (i64)c.sm_count * (per_sm > 0 ? per_sm : 1);
    if (n_host >= 0 && n_host < grid) grid = n_host > 0 ? n_host : 1;
    k<<<(int)grid, THREADS, smem, c.stream>>>(c.tab.perm, c.ctl, cls, slot, A, B, c.tab.cnt, rowptr, Ccrd, (T*)Cval);
    ++c.launches;
    return cudaGetLastError();
}

template <typename T, int CAP, int THREADS>
static cudaError_t launch_cap(const LaunchCtx& c, bool numeric, int cls, int n_host, const Csr& A, const Csr& B,
                              const i64* rowptr, int* Ccrd, void* Cval) {
    // 32-bit packed words when (column, slot) fits below the all-ones sentinel
    const bool narrow = (i64)B.ncols < (1ll << (32 - Log2<CAP>::value));
    if (narrow)
        return numeric ? launch_k<T, unsigned, CAP, THREADS, true>(c, cls, n_host, A, B, rowptr, Ccrd, Cval)
                       : launch_k<T, unsigned, CAP, THREADS, false>(c, cls, n_host, A, B, rowptr, Ccrd, Cval);
    return numeric ? launch_k<T, u64, CAP, THREADS, true>(c, cls, n_host, A, B, rowptr, Ccrd, Cval)
                   : launch_k<T, u64, CAP, THREADS, false>(c, cls, n_host, A, B, rowptr, Ccrd, Cval);
}

template <typename T>
static cudaError_t launch_t(const LaunchCtx& c, bool numeric, int cls, int n_host, const Csr& A, const Csr& B,
                            const i64* rowptr, int* Ccrd, void* Cval) {
    // the full class is launched for the largest row it actually holds when that is known: a
    // smaller accumulation array means more CTAs per SM and cheaper barriers
    int cap = (cls == CLS_ISM_SMEM_S) ? c.prm.smem_small_cap : c.prm.smem_cap;
    if (cls == CLS_ISM_SMEM && c.max_ub_smem > 0 && c.max_ub_smem < cap) cap = (int)c.max_ub_smem;
    if (cap <= 64) return launch_cap<T, 64, 64>(c, numeric, cls, n_host, A, B, rowptr, Ccrd, Cval);
    if (cap <= 256) return launch_cap<T, 256, 64>(c, numeric, cls, n_host, A, B, rowptr, Ccrd, Cval);
    if (cap <= 1024) return launch_cap<T, 1024, 128>(c, numeric, cls, n_host, A, B, rowptr, Ccrd, Cval);
    return launch_cap<T, 4096, 256>(c, numeric, cls, n_host, A, B, rowptr, Ccrd, Cval);
}

cudaError_t launch_ism_smem(const LaunchCtx& c, bool numeric, int cls, int n_host, const Csr& A, const Csr& B,
                            const i64* rowptr, int* Ccrd, void* Cval) {
    return c.is_f64 ? launch_t<double>(c, numeric, cls, n_host, A, B, rowptr, Ccrd, Cval)
                    : launch_t<float>(c, numeric, cls, n_host, A, B, rowptr, Ccrd, Cval);
}

}  // namespace spws
