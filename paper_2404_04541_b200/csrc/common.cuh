// Shared device-side definitions of the spws kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace spws {

typedef long long i64;
typedef unsigned long long u64;

constexpr int NCLASS = 13;
// Row classes = the workspace a row (or (i,j) fibre) is routed to in the symbolic pass.
enum RowClass : int {
    CLS_EMPTY = 0,      // no intermediate product
    CLS_ISM_REG8 = 1,   // insert-sort-merge in registers, 8 lanes per row (<= 8 products)
    CLS_ISM_REG16 = 2,  // ... 16 lanes per row (<= 16 products)
    CLS_ISM_REG = 3,    // ... one warp per row (<= 32 products)
    CLS_ISM_SMEM_S = 4, // insert-sort-merge in shared memory, small CTA
    CLS_ISM_SMEM = 5,   // insert-sort-merge in shared memory, full CTA
    CLS_DENSE_WARP = 6, // dense workspace (occupancy bitmap), one warp per row
    CLS_DENSE_HUB = 7,  // dense workspace, one CTA per row, heaviest rows (scheduled first)
    CLS_DENSE_CTA = 8,  // dense workspace, one CTA per row
    CLS_ISM_GLOBAL = 9, // accumulation array in shared memory, all array in global memory
    CLS_HASH_S = 10,    // hash table in shared memory (reduction at insert time), small CTA
    CLS_HASH = 11,      // hash table in shared memory, full CTA
    CLS_COPY8 = 12      // one A entry picking a B row of at most 8 entries: the result is that row, scaled
};
constexpr int NUM_SLOT = 16;   // work_counter[cls] in the symbolic pass, work_counter[NUM_SLOT + cls] in the numeric pass
constexpr int CEIL_SLOT = 32;  // work_counter[CEIL_SLOT + cls] in the gather-only (iteration-only) kernels
constexpr int EMIT_SLOT = 48;  // work_counter slot of the coordinate emission of the CTA dense route
constexpr int BW_SLOT = 49;    // work_counter slot of the word-list build
constexpr int N_WORK_COUNTERS = 64;
// index of a class in the public statistics (the three register classes are reported as one)
__host__ __device__ inline int public_class(int cls) { return cls == 0 ? 0 : ((cls <= 3 || cls == 12) ? 1 : cls - 2); }
constexpr int N_PUBLIC_CLASS = 10;
constexpr int HASH_SMALL_CAP = 1024;       // products of a row the small / the full hash workspace takes
constexpr int HASH_CAP = 4096;

// Capacities fixed at compile time.
constexpr int DENSE_WARP_BM_WORDS = 1024;  // bitmap words a warp-per-row workspace may span (32768 columns)
constexpr int DENSE_WARP_ACC = 256;        // outputs a warp-per-row numeric workspace may hold
constexpr int DENSE_WARP_MAX_UB = 4096;    // products a single warp is given at most
constexpr i64 DENSE_HUB_UB = 1ll << 17;    // rows with at least this many products are scheduled first
constexpr int DENSE_MAX_SPAN_WORDS = 16384;// 2^19 columns: the widest bitmap (8 bytes per word with its rank) one CTA holds
// Word lists of long B rows (symbolic pass of the CTA dense route): a B row with at least
// BW_MIN_LEN entries whose entries share bitmap words is also kept as (word index, bits) pairs,
// so that a row that picks it sets one word per pair instead of one bit per entry.
constexpr int LONG_A_ROW = 1024;     // entries of an A row beyond which a whole CTA computes its bounds
constexpr int BW_MIN_LEN = 256;
constexpr i64 BW_MAX_NNZ = 1ll << 26;      // lists are built only for a B with at most this many entries

enum DevStatus : int {
    DEV_OK = 0,
    DEV_NONCANONICAL = 4,
    DEV_SCRATCH_TOO_SMALL = 5,
    DEV_WORKSPACE_TOO_LARGE = 6,
    DEV_INTERNAL_OVERFLOW = 8
};

// Control block at the start of the scratch buffer (zeroed when a symbolic pass starts).
struct DevCtl {
    i64 nnz;
    i64 products;
    i64 max_ub;
    i64 max_ub_global;      // largest product count among CLS_ISM_GLOBAL rows
    i64 max_ub_smem;        // largest product count among CLS_ISM_SMEM rows (sizes that kernel's launch)
    i64 kept[2];            // TTM: surviving slices (level 0) and fibres (level 1)
    u64 bm_words_used;      // words handed out of the bitmap arena
    int status;
    int n_units;            // numeric dense CTA units (row, rank range)
    int n_warp_rows;        // numeric dense warp rows
    int max_span_words;     // widest bitmap among the dense rows
    int max_warp_cnt;       // most outputs of a row the warp numeric kernel takes
    int n_long;             // B rows with at least BW_MIN_LEN entries (candidates for a word list)
    int n_long_a;           // rows of A with more than LONG_A_ROW entries, left to the bounds kernel for long rows
    int class_count[NCLASS];
    int class_cursor[NCLASS];
    int work_counter[N_WORK_COUNTERS];   // dynamic work distribution; cleared before each pass
    i64 class_products[NCLASS];
    i64 class_nnz[NCLASS];
    i64 dense_warp_products, dense_warp_nnz;   // share of the dense rows the warp numeric kernel takes
};

struct ClassParams {
    int policy;             // spws_policy_t
    int reg_cap;            // CLS_ISM_REG: products <= reg_cap
    int smem_small_cap;     // CLS_ISM_SMEM_S
    int smem_cap;           // CLS_ISM_SMEM
    int unit_outputs;       // accumulator capacity of a dense CTA unit
    int max_span_words;     // dense allowed up to this many bitmap words
    float span_words_per_product;
    int unit_cap;           // entries available in the unit table
    u64 bm_arena_words;     // capacity of the bitmap arena
};

struct Csr {
    const i64* pos;
    const int* crd;
    const void* val;
    int nrows;
    int ncols;
};

// A CSF 3-tensor on the device (three compressed levels).
struct Csf3Dev {
    const i64* pos1;    // n0 + 1
    const i64* pos2;    // n1 + 1
    const int* crd0;
    const int* crd1;
    const int* crd2;
    const void* val;
    int n0, n1;
    i64 nnz;
};

// Per-row tables in scratch.
struct RowTables {
    i64* ub;
    int* cnt;
    int* jmin;
    int* jmax;
    unsigned char* cls;
    int* perm;
    i64* bm_off;        // word offset of the row's bitmap in the arena (dense classes)
    unsigned* bm_arena;
    int* warp_rows;     // numeric: rows handled by the warp-per-row dense kernel
    int* row_unit0;     // numeric: first CTA unit of a row
    int* unit_row;      // numeric: row of a CTA unit
};

// Products one dense CTA unit should take: 2^16 (measured on the power-law workload: units of
// 2^17 products cost the accumulation kernel 10 % more, of 2^18 products 35 % more), or more
// when the whole job is so large that the unit table (rows + 2^19 entries) would not hold that
// many units.
__host__ __device__ inline i64 dense_unit_products(i64 total_products) {
    const i64 need = (total_products + (1ll << 19) - 1) >> 19;
    return need > (1ll << 16) ? need : (1ll << 16);
}
__host__ __device__ inline int dense_units_of_row(i64 ub, i64 unit_products) {
    const i64 n = (ub + unit_products - 1) / unit_products;
    return (int)(n < 1 ? 1 : n);
}

__device__ __forceinline__ void raise_status(DevCtl* ctl, int s) { atomicCAS(&ctl->status, 0, s); }

// Rows of class `cls` are perm[off, off + n).
__device__ __forceinline__ void class_range(const DevCtl* ctl, int cls, int& off, int& n) {
    off = 0;
    for (int c = 0; c < cls; ++c) off += ctl->class_count[c];
    n = ctl->class_count[cls];
}

__device__ __forceinline__ int warp_incl_scan(int v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += t;
    }
    return v;
}

// Exclusive scan over a block of THREADS threads; `ws` needs 33 ints; every thread gets `total`.
template <int THREADS>
__device__ __forceinline__ int block_excl_scan(int v, int* ws, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int incl = warp_incl_scan(v);
    __syncthreads();                       // ws may still be read from a previous call
    if (lane == 31) ws[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int s = (lane < THREADS / 32) ? ws[lane] : 0;
        const int si = warp_incl_scan(s);
        if (lane < THREADS / 32) ws[lane] = si - s;
        if (lane == 31) ws[32] = si;
    }
    __syncthreads();
    total = ws[32];
    return ws[warp] + incl - v;
}

// First position in crd[lo, hi) whose coordinate is >= c (rows are sorted).
__device__ __forceinline__ i64 lower_bound_crd(const int* __restrict__ crd, i64 lo, i64 hi, i64 c) {
    while (lo < hi) {
        const i64 mid = (lo + hi) >> 1;
        if ((i64)__ldg(crd + mid) < c) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// Products are formed as a rounded multiply followed by rounded adds (no contraction), so the
// routes that sum in product order reproduce a plain sequential sum bit for bit.
__device__ __forceinline__ double mul_rn(double a, double b) { return __dmul_rn(a, b); }
__device__ __forceinline__ float mul_rn(float a, float b) { return __fmul_rn(a, b); }
__device__ __forceinline__ double add_rn(double a, double b) { return __dadd_rn(a, b); }
__device__ __forceinline__ float add_rn(float a, float b) { return __fadd_rn(a, b); }

// ---- launchers (defined in the .cu files) ------------------------------------------------
struct LaunchCtx {
    cudaStream_t stream;
    int sm_count;
    DevCtl* ctl;
    ClassParams prm;
    RowTables tab;
    int is_f64;
    int dense_smem_words;    // bitmap words the CTA dense kernels reserve (from ncols)
    char* rest;              // scratch after the fixed tables: bitmap arena, then the ISM-global arena
    size_t rest_bytes;
    int global_cap;          // accumulation-array capacity of CLS_ISM_GLOBAL
    i64 max_ub_smem;         // largest product count of a CLS_ISM_SMEM row when known (0: unknown)
    uint2* bw;               // word lists of long B rows, indexed like B's entries (null: not built)
    int* bw_long;            // the long B rows, in arrival order
    int bw_long_cap;
    int4* brow;                 // per B row: first column, last column, length (null: not kept)
    mutable int launches;    // kernels enqueued through this context
};

// setup.cu
cudaError_t launch_validate(const LaunchCtx& c, const Csr& A, const Csr& B, i64 nnzA, i64 nnzB);
cudaError_t launch_row_bounds(const LaunchCtx& c, const Csr& A, const Csr& B, i64 nnzA);
cudaError_t launch_bw_build(const LaunchCtx& c, const Csr& B);
cudaError_t launch_bin_rows(const LaunchCtx& c, int m);
cudaError_t launch_dense_rebin(const LaunchCtx& c, int m, const i64* rowptr);
cudaError_t launch_class_nnz(const LaunchCtx& c, int m);
// as_flags: scan (cnt[i] > 0) instead of cnt[i]
cudaError_t launch_scan_counts(const LaunchCtx& c, const int* cnt, int n, i64* out, i64* block_sums, i64* total_out, bool as_flags = false);
cudaError_t launch_ttm_scan_compact(const LaunchCtx& c, int n_i, int n_ij, const i64* Apos1, const int* Acrd0, const int* Acrd1,
                                    i64* rowptr_raw, i64* fpos, int* sflags, i64* spos, i64* block_sums, i64* nnz_out,
                                    i64* Cpos0, int* Ccrd0, i64* Cpos1, int* Ccrd1, i64* Cpos2);
// class kernels: n_host < 0 means "size the grid for any count"
cudaError_t launch_ism_reg(const LaunchCtx& c, bool numeric, int cls, int n_host, const Csr& A, const Csr& B,
                           const i64* rowptr, int* Ccrd, void* Cval);
cudaError_t launch_ism_smem(const LaunchCtx& c, bool numeric, int cls, int n_host, const Csr& A, const Csr& B,
                            const i64* rowptr, int* Ccrd, void* Cval);
cudaError_t launch_dense_sym_warp(const LaunchCtx& c, const Csr& A, const Csr& B);
cudaError_t launch_dense_sym_cta(const LaunchCtx& c, const Csr& A, const Csr& B);
// chk_idx / chk_val non-null: the gather-only form of the same kernel (workspace stripped, checksums out)
cudaError_t launch_dense_num_warp(const LaunchCtx& c, int n_host, int max_span_words, int max_cnt, const Csr& A, const Csr& B,
                                  const i64* rowptr, int* Ccrd, void* Cval, u64* chk_idx = nullptr, double* chk_val = nullptr);
// phase 0: write the coordinates and clear the value segments several units add into; 1: accumulate
cudaError_t launch_dense_num_cta(const LaunchCtx& c, int phase, int n_units_host, int max_span_words, i64 total_products,
                                 const Csr& A, const Csr& B, const i64* rowptr, int* Ccrd, void* Cval,
                                 u64* chk_idx = nullptr, double* chk_val = nullptr);
cudaError_t launch_ism_global(const LaunchCtx& c, bool numeric, int n_host, const Csr& A, const Csr& B,
                              const i64* rowptr, int* Ccrd, void* Cval);
cudaError_t launch_hash(const LaunchCtx& c, bool numeric, int cls, int n_host, const Csr& A, const Csr& B, const i64* rowptr,
                        int* Ccrd, void* Cval);

// outer.cu: second-order workspaces of the outer-product form
cudaError_t launch_outer_counts(const LaunchCtx& c, const Csr& At, const Csr& B, int* cnt);
size_t outer_sort_scratch_bytes(i64 n);
cudaError_t launch_outer_ism(const LaunchCtx& c, bool numeric, const Csr& At, const Csr& B, const i64* koff, i64 P, i64 cap, i64 J,
                             int label_bits, u64* kA, void* vA, u64* kB, void* vB, int* head, i64* at, char* sort_tmp,
                             i64* block_sums, i64* nnz_dev, i64* nnz_host_pinned, bool* result_first);
cudaError_t launch_coo_pos(const LaunchCtx& c, const u64* ukeys, i64 nnz, i64 m, i64 J, i64* pos);
cudaError_t launch_coo_out(const LaunchCtx& c, const u64* ukeys, const void* uvals, i64 nnz, i64 J, int* Ccrd, void* Cval);
cudaError_t launch_outer_dense(const LaunchCtx& c, bool numeric, const Csr& At, const Csr& B, const i64* koff, i64 P, i64 m, i64 J,
                               unsigned* dbits, void* dvals, int* cnt, const i64* pos, int* Ccrd, void* Cval);
cudaError_t launch_outer_total(const LaunchCtx& c, const Csr& At, const Csr& B, u64* total_mapped_host);
// higher.cu: the higher-order scatters with coordinate-form output
cudaError_t launch_higher_total(const LaunchCtx& c, int form, const Csf3Dev& B, const Csr& C, u64* total_mapped_host);
cudaError_t launch_higher_setup(const LaunchCtx& c, int form, const Csf3Dev& B, const Csr& C, int* fib_of, int* slice_of, int* cnt);
cudaError_t launch_higher_ism(const LaunchCtx& c, bool numeric, int form, const Csf3Dev& B, const Csr& C, const Csr& D, const int* fib_of,
                              const int* slice_of, const i64* eoff, i64 P, i64 cap, u64 d1, u64 d2, int label_bits, u64* kA, void* vA,
                              u64* kB, void* vB, int* head, i64* at, char* sort_tmp, i64* block_sums, i64* nnz_dev,
                              i64* nnz_host_pinned, bool* result_first);
cudaError_t launch_higher_unpack(const LaunchCtx& c, int order, const u64* ukeys, const void* uvals, i64 nnz, u64 d1, u64 d2, int* o0,
                                 int* o1, int* o2, void* oval);

}  // namespace spws
