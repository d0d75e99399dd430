// C ABI of the spws library: handles, plans, expression check, scratch layout and the launch
// sequences of the symbolic and numeric passes.  Host code only.
#include <algorithm>
#include <cctype>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/spws.h"
#include "common.cuh"

using namespace spws;

struct spws_handle_s {
    cudaStream_t stream = nullptr;
    int device = 0;
    int sm_count = 0;
};

struct spws_plan_s {
    spws_handle_t h = nullptr;
    int kind = 0;               // 0 SpGEMM (CSR x CSR -> CSR), 1 TTM (CSF3 x CSR -> CSF3), 2 outer-product SpGEMM (A by rows k)
    int is_f64 = 1;
    int policy = SPWS_AUTO;
    spws_options_t opt{};
    DevCtl* host_ctl = nullptr; // pinned
    bool symbolic_ok = false;
    spws_stats_t stats{};
    // what the last symbolic pass saw (numeric must be called with the same shapes and scratch)
    int64_t m = 0;
    void* scratch = nullptr;
    int max_span_words = 0;     // widest dense bitmap of the last symbolic pass
    int max_warp_cnt = 0;       // most outputs of a warp-numeric row
    int64_t max_ub_smem = 0;    // most products of a shared-memory ISM row
    int64_t bin_rows[NCLASS] = {};  // rows per internal class of the last symbolic pass
    // outer-product form: what the last symbolic pass decided
    int64_t outer_products = 0;
    bool outer_dense = false;
    // optional per-kernel timing: ev[g] is recorded after group g; ev_start[] before each pass
    bool profiling = false;
    cudaEvent_t ev[SPWS_T_COUNT] = {};
    cudaEvent_t ev_start[3] = {};
    bool ev_ran[SPWS_T_COUNT] = {};
    bool ev_pass[3] = {};
};

namespace {

inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
// int64_t is `long` on this ABI, the kernels use `long long`: same width, distinct types
inline i64* LL(int64_t* p) { return reinterpret_cast<i64*>(p); }
inline const i64* LL(const int64_t* p) { return reinterpret_cast<const i64*>(p); }

// ---- expression -------------------------------------------------------------------------
struct Access { std::string name; std::vector<std::string> idx; };

bool parse_access(const char*& s, Access& a) {
    while (*s && isspace((unsigned char)*s)) ++s;
    if (!(isalpha((unsigned char)*s) || *s == '_')) return false;
    while (isalnum((unsigned char)*s) || *s == '_') a.name.push_back(*s++);
    while (*s && isspace((unsigned char)*s)) ++s;
    if (*s != '(') return false;
    ++s;
    for (;;) {
        while (*s && isspace((unsigned char)*s)) ++s;
        std::string v;
        if (!(isalpha((unsigned char)*s) || *s == '_')) return false;
        while (isalnum((unsigned char)*s) || *s == '_') v.push_back(*s++);
        a.idx.push_back(v);
        while (*s && isspace((unsigned char)*s)) ++s;
        if (*s == ',') { ++s; continue; }
        if (*s == ')') { ++s; break; }
        return false;
    }
    while (*s && isspace((unsigned char)*s)) ++s;
    return true;
}

bool distinct(const std::vector<std::string>& v) {
    for (size_t a = 0; a < v.size(); ++a)
        for (size_t b = a + 1; b < v.size(); ++b)
            if (v[a] == v[b]) return false;
    return true;
}

// Accepts (kind in brackets)
//   [0, 1] out(o_1..o_N) = x(o_1..o_{N-1}, r) * y(r, o_N), N = 2 or 3, formats (CSR, CSR, CSR) or
//     (CSF3, CSF3, CSR): loop order o_1 -> .. -> r -> o_N against output order o_1 -> .. -> o_N: the
//     reduction variable sits one position from the innermost index: a first-order scatter;
//   [2] out(o_1, o_2) = x(r, o_1) * y(r, o_2), formats (CSR, CSR, CSR): loop order r -> o_1 -> o_2, both
//     output indices scatter: a second-order scatter (the outer-product form);
//   [3] out(o_1, o_2, o_3) = x(r, o_1, o_2) * y(r, o_3), formats (COO, CSF3, CSR): third-order scatter;
//   [4] out(o_1, o_2, o_3) = x(o_1, r, o_2) * y(r, o_3), formats (COO, CSF3, CSR): o_1 is shared by the
//     loop nest and the output, the other two indices scatter;
//   [5] out(o_1, o_2) = x(r_1, r_2, o_1) * y(r_1, o_2) * z(r_2, o_2), formats (COO, CSF3, CSR, CSR): two
//     reduction variables outermost, a second-order scatter.
// Returns the kind or -1; `n_fmts` is 3 (two operands) or 4 (three operands).
int classify_expression(const char* expr, const spws_format_t* fmts, int n_fmts) {
    const char* s = expr;
    Access out, x, y, z;
    if (!parse_access(s, out)) return -1;
    if (*s == '+' && s[1] == '=') s += 2; else if (*s == '=') s += 1; else return -1;
    if (!parse_access(s, x)) return -1;
    if (*s != '*') return -1;
    ++s;
    if (!parse_access(s, y)) return -1;
    int n_ops = 2;
    if (*s == '*') {
        ++s;
        if (!parse_access(s, z)) return -1;
        n_ops = 3;
    }
    if (*s != '\0') return -1;
    if (n_ops + 1 != n_fmts) return -1;
    const size_t N = out.idx.size();
    if (N != 2 && N != 3) return -1;
    if (!distinct(out.idx) || !distinct(x.idx) || !distinct(y.idx) || y.idx.size() != 2) return -1;
    if (out.name == x.name || out.name == y.name || (n_ops == 3 && (out.name == z.name || !distinct(z.idx) || z.idx.size() != 2))) return -1;
    auto is_output = [&](const std::string& v) { for (const auto& o : out.idx) if (o == v) return true; return false; };
    if (n_ops == 3) {
        if (N != 2 || x.idx.size() != 3) return -1;
        const std::string &r1 = x.idx[0], &r2 = x.idx[1];
        if (is_output(r1) || is_output(r2) || r1 == r2) return -1;
        if (x.idx[2] != out.idx[0] || y.idx[0] != r1 || y.idx[1] != out.idx[1] || z.idx[0] != r2 || z.idx[1] != out.idx[1]) return -1;
        if (fmts[0] != SPWS_COO || fmts[1] != SPWS_CSF3 || fmts[2] != SPWS_CSR || fmts[3] != SPWS_CSR) return -1;
        return 5;
    }
    if (x.idx.size() != N) return -1;
    if (fmts[0] == SPWS_COO) {
        if (N != 3 || fmts[1] != SPWS_CSF3 || fmts[2] != SPWS_CSR) return -1;
        if (!is_output(x.idx[0]) && x.idx[1] == out.idx[0] && x.idx[2] == out.idx[1] && y.idx[0] == x.idx[0] && y.idx[1] == out.idx[2]) return 3;
        if (!is_output(x.idx[1]) && x.idx[0] == out.idx[0] && x.idx[2] == out.idx[1] && y.idx[0] == x.idx[1] && y.idx[1] == out.idx[2]) return 4;
        return -1;
    }
    if (N == 2 && x.idx[0] == y.idx[0] && x.idx[1] == out.idx[0] && y.idx[1] == out.idx[1] && !is_output(x.idx[0])) {
        if (fmts[0] != SPWS_CSR || fmts[1] != SPWS_CSR || fmts[2] != SPWS_CSR) return -1;
        return 2;
    }
    const std::string& r = x.idx[N - 1];
    if (is_output(r)) return -1;                                             // r must be a reduction variable
    for (size_t a = 0; a + 1 < N; ++a) if (x.idx[a] != out.idx[a]) return -1;
    if (y.idx[0] != r || y.idx[1] != out.idx[N - 1]) return -1;
    if (N == 2) {
        if (fmts[0] != SPWS_CSR || fmts[1] != SPWS_CSR || fmts[2] != SPWS_CSR) return -1;
        return 0;
    }
    if (fmts[0] != SPWS_CSF3 || fmts[1] != SPWS_CSF3 || fmts[2] != SPWS_CSR) return -1;
    return 1;
}

bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

// ---- scratch layout ------------------------------------------------------------------------
struct Layout {
    size_t ctl, ub, rowptr_raw, cnt, jmin, jmax, cls, perm, bm_off, warp_rows, row_unit0, unit_row, block_sums,
        fpos, sflags, spos, bw_long, bw, brow, rest, fixed_end;
    bool has_brow;
    int unit_cap;
    int bw_long_cap;            // 0: no word lists for this B
    int dense_smem_words;
};

Layout make_layout(const spws_plan_s* p, int64_t m, int64_t ncols, int64_t n_i, int64_t nnzB, int64_t k, int64_t nnzA) {
    Layout L{};
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align256(o + bytes); return at; };
    L.ctl = take(sizeof(DevCtl));
    L.ub = take(8 * (size_t)m);
    L.rowptr_raw = take(8 * ((size_t)m + 1));
    L.cnt = take(4 * (size_t)m);
    L.jmin = take(4 * (size_t)m);
    L.jmax = take(4 * (size_t)m);
    L.cls = take((size_t)m);
    L.perm = take(4 * (size_t)m);
    L.bm_off = take(8 * (size_t)m);
    L.warp_rows = take(4 * (size_t)m);
    L.row_unit0 = take(4 * (size_t)m);
    // one unit per dense row plus at most 2^19 more for rows split by product count
    const int64_t span_cap = ncols < p->opt.dense_max_span ? ncols : p->opt.dense_max_span;
    int64_t ucap = m + (1ll << 19) + 1024;
    if (ucap > 0x7fff0000ll) ucap = 0x7fff0000ll;
    L.unit_cap = (int)ucap;
    L.unit_row = take(4 * (size_t)ucap);
    int64_t words = (span_cap + 31) / 32 + 1;
    if (words > DENSE_MAX_SPAN_WORDS) words = DENSE_MAX_SPAN_WORDS;
    L.dense_smem_words = (int)((words + 7) & ~7ll);
    const size_t longest = (size_t)(m > n_i ? m : n_i);
    L.block_sums = take(16 * (longest / 2048 + 2));     // two arrays for the 3-tensor form's paired scan
    if (p->kind == 1) {
        L.fpos = take(8 * ((size_t)m + 1));
        L.sflags = take(4 * (size_t)n_i);
        L.spos = take(8 * ((size_t)n_i + 1));
    }
    // word lists of long B rows (dense routes): one 8-byte slot per entry of B, used only at the
    // positions of rows with at least BW_MIN_LEN entries
    if (p->policy != SPWS_SPARSE_ISM && p->policy != SPWS_HASH && nnzB >= BW_MIN_LEN && nnzB <= BW_MAX_NNZ) {
        L.bw_long_cap = (int)(nnzB / BW_MIN_LEN + 1);
        L.bw_long = take(4 * (size_t)L.bw_long_cap);
        L.bw = take(8 * (size_t)nnzB);
    }
    // first column, last column and length of every B row, for the bounds kernel: kept when A
    // picks every B row several times over on average
    if (k > 0 && nnzA >= 4 * k) {
        L.has_brow = true;
        L.brow = take(16 * (size_t)k);
    }
    L.fixed_end = o;
    L.rest = o;
    return L;
}

// All-array slots the global-memory ISM is given: one per CTA it can keep busy (two per SM), but
// no more than rows of that class and no more than fit 2 GiB; eight at least.
size_t global_ism_slots(const spws_plan_s* p, size_t slot_bytes, int64_t rows) {
    size_t slots = 2 * (size_t)p->h->sm_count;
    const size_t fit = slot_bytes ? ((size_t)2 << 30) / slot_bytes : slots;
    if (slots > fit) slots = fit;
    if (slots < 8) slots = 8;
    if ((int64_t)slots > rows) slots = (size_t)(rows > 0 ? rows : 1);
    return slots;
}

// what follows the fixed tables: one bitmap per row in the worst case (dense routes), and room
// for the all-array slots of the global-memory ISM at min(ncols, 2^22) components each
size_t rest_reserve(const spws_plan_s* p, int64_t m, int64_t ncols) {
    size_t bytes = 0;
    if (p->policy != SPWS_SPARSE_ISM && p->policy != SPWS_HASH) {
        const int64_t span_cap = ncols < p->opt.dense_max_span ? ncols : p->opt.dense_max_span;
        const size_t nw = (size_t)((span_cap + 31) / 32 + 1);
        bytes += align256((size_t)m * ((nw + (nw + 31) / 32 + 3) & ~(size_t)3) * 4);
    }
    if (p->policy != SPWS_DENSE) {
        // global-memory ISM: eight slots of min(ncols, 2^22) components, and never less than the one
        // slot a row over all ncols columns needs in the numeric pass
        const int64_t elems = ncols < (1ll << 22) ? ncols : (1ll << 22);
        const size_t comp = 4 + (p->is_f64 ? 8 : 4);
        const size_t slot = align256(2 * (size_t)((elems + 63) & ~63ll) * comp);
        const size_t one_full = align256(2 * (size_t)((ncols + 63) & ~63ll) * comp);
        const size_t many = slot * global_ism_slots(p, slot, 0x7fffffff);
        bytes += many > one_full ? many : one_full;
    }
    return bytes;
}

struct Shapes {
    int64_t m, k, ncols, nnzA, nnzB, n_i;
    Csr A, B;
};

spws_status_t check_operands(const spws_plan_s* p, const spws_tensor_t* A, const spws_tensor_t* B, Shapes& S,
                             bool need_pointers = true) {
    if (!A || !B) return SPWS_INVALID_ARGUMENT;
    if (B->order != 2) return SPWS_INVALID_ARGUMENT;
    if (p->kind == 0) {
        if (A->order != 2) return SPWS_INVALID_ARGUMENT;
        S.m = A->dims[0]; S.k = A->dims[1]; S.nnzA = A->n[1]; S.n_i = 0;
        S.A = Csr{LL(A->pos[1]), A->crd[1], A->val, (int)S.m, (int)S.k};
    } else if (p->kind == 2) {                  // A stored by its rows k: dims = (K, I)
        if (A->order != 2) return SPWS_INVALID_ARGUMENT;
        S.m = A->dims[1]; S.k = A->dims[0]; S.nnzA = A->n[1]; S.n_i = 0;
        S.A = Csr{LL(A->pos[1]), A->crd[1], A->val, (int)S.k, (int)S.m};
    } else {
        if (A->order != 3) return SPWS_INVALID_ARGUMENT;
        S.m = A->n[1]; S.k = A->dims[2]; S.nnzA = A->n[2]; S.n_i = A->n[0];
        S.A = Csr{LL(A->pos[2]), A->crd[2], A->val, (int)S.m, (int)S.k};
        if (A->n[0] < 0 || A->n[0] > A->dims[0] || A->n[1] < A->n[0]) return SPWS_INVALID_ARGUMENT;
    }
    S.ncols = B->dims[1];
    S.nnzB = B->n[1];
    S.B = Csr{LL(B->pos[1]), B->crd[1], B->val, (int)B->dims[0], (int)S.ncols};
    if (S.m < 0 || S.k < 0 || S.ncols < 0 || S.nnzA < 0 || S.nnzB < 0) return SPWS_INVALID_ARGUMENT;
    if (S.m > 0x7ffffff0ll || S.k > 0x7ffffff0ll || S.ncols > 0x7ffffff0ll || B->dims[0] > 0x7ffffff0ll)
        return SPWS_INVALID_ARGUMENT;
    if (S.k != B->dims[0]) return SPWS_DIM_MISMATCH;
    if (!need_pointers) return SPWS_OK;
    if ((p->kind == 2 ? S.k : S.m) > 0 && (!S.A.pos)) return SPWS_INVALID_ARGUMENT;
    if (S.nnzA > 0 && (!S.A.crd || !S.A.val)) return SPWS_INVALID_ARGUMENT;
    if (B->dims[0] > 0 && !S.B.pos) return SPWS_INVALID_ARGUMENT;
    if (S.nnzB > 0 && (!S.B.crd || !S.B.val)) return SPWS_INVALID_ARGUMENT;
    return SPWS_OK;
}

spws_status_t check_output_dims(const spws_plan_s* p, const spws_tensor_t* A, const spws_tensor_t* B, const spws_tensor_t* C) {
    if (!C) return SPWS_INVALID_ARGUMENT;
    if (p->kind == 0 || p->kind == 2) {
        if (C->order != 2) return SPWS_INVALID_ARGUMENT;
        if (C->dims[0] != A->dims[p->kind == 0 ? 0 : 1] || C->dims[1] != B->dims[1]) return SPWS_DIM_MISMATCH;
        if (!C->pos[1]) return SPWS_INVALID_ARGUMENT;
    } else {
        if (C->order != 3) return SPWS_INVALID_ARGUMENT;
        if (C->dims[0] != A->dims[0] || C->dims[1] != A->dims[1] || C->dims[2] != B->dims[1]) return SPWS_DIM_MISMATCH;
        if (!C->pos[0] || !C->pos[1] || !C->pos[2]) return SPWS_INVALID_ARGUMENT;
        if (A->n[0] > 0 && !C->crd[0]) return SPWS_INVALID_ARGUMENT;
        if (A->n[1] > 0 && !C->crd[1]) return SPWS_INVALID_ARGUMENT;
    }
    return SPWS_OK;
}

LaunchCtx make_ctx(const spws_plan_s* p, char* scratch, size_t scratch_bytes, const Layout& L) {
    LaunchCtx c{};
    c.stream = p->h->stream;
    c.sm_count = p->h->sm_count;
    c.ctl = reinterpret_cast<DevCtl*>(scratch + L.ctl);
    c.prm.policy = p->policy;
    c.prm.reg_cap = p->opt.ism_warp_cap;
    c.prm.smem_cap = p->opt.ism_cta_cap;
    c.prm.smem_small_cap = p->opt.ism_cta_cap >= 1024 ? 256 : (p->opt.ism_cta_cap >= 256 ? 64 : p->opt.ism_cta_cap);
    c.prm.unit_outputs = p->opt.dense_unit_outputs;
    c.prm.max_span_words = (p->opt.dense_max_span + 31) / 32;
    c.prm.span_words_per_product = p->opt.dense_span_words_per_product;
    c.prm.unit_cap = L.unit_cap;
    c.rest = scratch + L.rest;
    c.rest_bytes = scratch_bytes > L.rest ? scratch_bytes - L.rest : 0;
    c.prm.bm_arena_words = (p->policy == SPWS_SPARSE_ISM || p->policy == SPWS_HASH) ? 0 : c.rest_bytes / 4;
    c.dense_smem_words = L.dense_smem_words;
    c.tab.ub = reinterpret_cast<i64*>(scratch + L.ub);
    c.tab.cnt = reinterpret_cast<int*>(scratch + L.cnt);
    c.tab.jmin = reinterpret_cast<int*>(scratch + L.jmin);
    c.tab.jmax = reinterpret_cast<int*>(scratch + L.jmax);
    c.tab.cls = reinterpret_cast<unsigned char*>(scratch + L.cls);
    c.tab.perm = reinterpret_cast<int*>(scratch + L.perm);
    c.tab.bm_off = reinterpret_cast<i64*>(scratch + L.bm_off);
    c.tab.bm_arena = reinterpret_cast<unsigned*>(scratch + L.rest);
    c.tab.warp_rows = reinterpret_cast<int*>(scratch + L.warp_rows);
    c.tab.row_unit0 = reinterpret_cast<int*>(scratch + L.row_unit0);
    c.tab.unit_row = reinterpret_cast<int*>(scratch + L.unit_row);
    c.is_f64 = p->is_f64;
    c.global_cap = p->opt.fallback_cap;
    if (L.bw_long_cap > 0) {
        c.bw = reinterpret_cast<uint2*>(scratch + L.bw);
        c.bw_long = reinterpret_cast<int*>(scratch + L.bw_long);
        c.bw_long_cap = L.bw_long_cap;
    }
    if (L.has_brow) c.brow = reinterpret_cast<int4*>(scratch + L.brow);
    return c;
}

spws_status_t from_dev_status(int s) {
    switch (s) {
        case DEV_OK: return SPWS_OK;
        case DEV_NONCANONICAL: return SPWS_NONCANONICAL_INPUT;
        case DEV_SCRATCH_TOO_SMALL: return SPWS_SCRATCH_TOO_SMALL;
        case DEV_WORKSPACE_TOO_LARGE: return SPWS_WORKSPACE_TOO_LARGE;
        default: return SPWS_INTERNAL_OVERFLOW;
    }
}

#define CUDA_TRY(x) do { if ((x) != cudaSuccess) { cudaGetLastError(); return SPWS_CUDA_ERROR; } } while (0)

inline void mark(spws_plan_s* p, int group) {
    if (!p->profiling) return;
    cudaEventRecord(p->ev[group], p->h->stream);
    p->ev_ran[group] = true;
}
// timing groups of pass 0 (symbolic), 1 (numeric), 2 (gather-only ceiling)
const int PASS_GROUPS[4] = {0, SPWS_T_NUM_ISM_REG, SPWS_T_CEIL_DENSE_WARP, SPWS_T_COUNT};

inline void mark_start(spws_plan_s* p, int pass) {
    if (!p->profiling) return;
    const int g0 = PASS_GROUPS[pass], g1 = PASS_GROUPS[pass + 1];
    for (int g = g0; g < g1; ++g) p->ev_ran[g] = false;
    cudaEventRecord(p->ev_start[pass], p->h->stream);
    p->ev_pass[pass] = true;
}

// ---- outer-product form (kind 2): scratch layout and the two passes -------------------------
struct OuterLayout {
    size_t ctl, cnt, koff, block_sums, fixed_end;
    // sparse workspace
    size_t kA, kB, vA, vB, head, at, sort_tmp, ism_end;
    // dense workspace
    size_t dbits, dvals, dcnt, dense_end;
    int64_t N;                  // entries of each (label, value) array
};

OuterLayout make_outer_layout(const spws_plan_s* p, int64_t I, int64_t K, int64_t J, int64_t P) {
    OuterLayout L{};
    const size_t V = p->is_f64 ? 8 : 4;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align256(o + bytes); return at; };
    const int64_t cap = p->opt.outer_cap > 0 ? p->opt.outer_cap : P;
    L.N = P + (cap < P ? cap : 0);
    const int64_t longest = std::max<int64_t>(std::max<int64_t>(K, I), L.N);
    L.ctl = take(sizeof(DevCtl));
    L.cnt = take(4 * (size_t)K);
    L.koff = take(8 * ((size_t)K + 1));
    L.block_sums = take(8 * ((size_t)longest / 2048 + 2));
    L.fixed_end = o;
    L.kA = take(8 * (size_t)L.N);
    L.kB = take(8 * (size_t)L.N);
    L.vA = take(V * (size_t)L.N);
    L.vB = take(V * (size_t)L.N);
    L.head = take(4 * (size_t)L.N);
    L.at = take(8 * ((size_t)L.N + 1));
    L.sort_tmp = take(outer_sort_scratch_bytes(L.N));
    L.ism_end = o;
    o = L.fixed_end;
    const size_t row_words = (size_t)((J + 31) / 32);
    L.dbits = take(4 * (size_t)I * row_words);
    L.dvals = take(V * (size_t)I * (size_t)J);
    L.dcnt = take(4 * (size_t)I);
    L.dense_end = o;
    return L;
}

int label_bits_of(int64_t I, int64_t J) {
    const unsigned long long top = (unsigned long long)I * (unsigned long long)J;
    int bits = 1;
    while (bits < 64 && (top >> bits) != 0) ++bits;
    return bits;
}

// products of the outer form, counted on the device into a word of the plan's pinned block
spws_status_t outer_count_products(spws_plan_s* p, const Shapes& S, int64_t* P) {
    LaunchCtx c{};
    c.stream = p->h->stream;
    c.sm_count = p->h->sm_count;
    u64* word = reinterpret_cast<u64*>(&p->host_ctl->products);
    *word = 0;
    CUDA_TRY(launch_outer_total(c, S.A, S.B, word));
    CUDA_TRY(cudaStreamSynchronize(c.stream));
    *P = (int64_t)*word;
    return SPWS_OK;
}

bool outer_wants_dense(const spws_plan_s* p, int64_t I, int64_t J, int64_t P, size_t scratch_bytes, const OuterLayout& L, spws_status_t* st) {
    *st = SPWS_OK;
    const bool fits = scratch_bytes >= L.dense_end;
    if (p->policy == SPWS_DENSE) {
        if (!fits) *st = SPWS_WORKSPACE_TOO_LARGE;
        return true;
    }
    if (p->policy == SPWS_SPARSE_ISM || p->policy == SPWS_HASH) return false;
    // measured on B200 (I = J = 10^4): the dense workspace wins from the smallest product count on,
    // so it is taken whenever it is small in absolute terms or next to the work
    return fits && ((double)I * (double)J <= 134217728.0 || (double)P * 16.0 >= (double)I * (double)J);
}

spws_status_t outer_symbolic(spws_plan_s* plan, const Shapes& S, spws_tensor_t* C, void* scratch, size_t scratch_bytes, int64_t* sizes_out) {
    const int64_t I = S.m, K = S.k, J = S.ncols;
    if (I * J < 0 || (I > 0 && J > (int64_t)(0x7fffffffffffffffll / (I > 0 ? I : 1)))) return SPWS_INVALID_ARGUMENT;
    int64_t P = 0;
    spws_status_t st = outer_count_products(plan, S, &P);
    if (st != SPWS_OK) return st;
    if (P > 0x7fff0000ll) return SPWS_INTERNAL_OVERFLOW;            // product ordinals and scans are 31-bit here
    const OuterLayout L = make_outer_layout(plan, I, K, J, P);
    if (scratch_bytes < L.fixed_end) return SPWS_SCRATCH_TOO_SMALL;
    const bool dense = outer_wants_dense(plan, I, J, P, scratch_bytes, L, &st);
    if (st != SPWS_OK) return st;
    if (!dense && scratch_bytes < L.ism_end) return SPWS_SCRATCH_TOO_SMALL;
    char* sc = static_cast<char*>(scratch);
    LaunchCtx c{};
    c.stream = plan->h->stream;
    c.sm_count = plan->h->sm_count;
    c.ctl = reinterpret_cast<DevCtl*>(sc + L.ctl);
    c.is_f64 = plan->is_f64;
    cudaStream_t stream = c.stream;
    CUDA_TRY(cudaMemsetAsync(c.ctl, 0, sizeof(DevCtl), stream));
    mark_start(plan, 0);
    int* cnt = reinterpret_cast<int*>(sc + L.cnt);
    i64* koff = reinterpret_cast<i64*>(sc + L.koff);
    i64* block_sums = reinterpret_cast<i64*>(sc + L.block_sums);
    CUDA_TRY(launch_outer_counts(c, S.A, S.B, cnt));
    CUDA_TRY(launch_scan_counts(c, cnt, (int)K, koff, block_sums, &c.ctl->products));
    mark(plan, SPWS_T_SYM_BOUNDS);
    i64* pos = LL(C->pos[1]);
    int64_t nnz = 0;
    if (dense) {
        const size_t row_words = (size_t)((J + 31) / 32);
        CUDA_TRY(cudaMemsetAsync(sc + L.dbits, 0, 4 * (size_t)I * row_words, stream));
        CUDA_TRY(launch_outer_dense(c, false, S.A, S.B, koff, P, I, J, reinterpret_cast<unsigned*>(sc + L.dbits), nullptr,
                                    reinterpret_cast<int*>(sc + L.dcnt), nullptr, nullptr, nullptr));
        CUDA_TRY(launch_scan_counts(c, reinterpret_cast<int*>(sc + L.dcnt), (int)I, pos, block_sums, &c.ctl->nnz));
        mark(plan, SPWS_T_SYM_DENSE_CTA);
    } else {
        bool first = true;
        i64* nnz_host = reinterpret_cast<i64*>(&plan->host_ctl->nnz);
        const int64_t cap = plan->opt.outer_cap > 0 ? plan->opt.outer_cap : (P > 0 ? P : 1);
        CUDA_TRY(launch_outer_ism(c, false, S.A, S.B, koff, P, cap, J, label_bits_of(I, J), reinterpret_cast<u64*>(sc + L.kA), nullptr,
                                  reinterpret_cast<u64*>(sc + L.kB), nullptr, reinterpret_cast<int*>(sc + L.head),
                                  reinterpret_cast<i64*>(sc + L.at), sc + L.sort_tmp, block_sums, &c.ctl->nnz, nnz_host, &first));
        nnz = *nnz_host;
        CUDA_TRY(cudaMemcpyAsync(&c.ctl->nnz, nnz_host, sizeof(i64), cudaMemcpyHostToDevice, stream));
        CUDA_TRY(launch_coo_pos(c, reinterpret_cast<u64*>(sc + (first ? L.kA : L.kB)), nnz, I, J, pos));
        mark(plan, SPWS_T_SYM_ISM_GLOBAL);
    }
    CUDA_TRY(cudaMemcpyAsync(plan->host_ctl, c.ctl, sizeof(DevCtl), cudaMemcpyDeviceToHost, stream));
    CUDA_TRY(cudaStreamSynchronize(stream));
    const DevCtl& hc = *plan->host_ctl;
    plan->stats = spws_stats_t{};
    plan->stats.device_status = hc.status;
    if (hc.status != 0) return from_dev_status(hc.status);
    plan->stats.rows = I;
    plan->stats.products = P;
    plan->stats.nnz = hc.nnz;
    plan->stats.rows_per_class[dense ? public_class(CLS_DENSE_CTA) : public_class(CLS_ISM_GLOBAL)] = I;
    plan->stats.products_per_class[dense ? public_class(CLS_DENSE_CTA) : public_class(CLS_ISM_GLOBAL)] = P;
    plan->stats.nnz_per_class[dense ? public_class(CLS_DENSE_CTA) : public_class(CLS_ISM_GLOBAL)] = hc.nnz;
    plan->stats.launches_symbolic = c.launches;
    plan->outer_products = P;
    plan->outer_dense = dense;
    C->n[0] = C->dims[0];
    C->n[1] = hc.nnz;
    C->n[2] = 0;
    if (sizes_out) { sizes_out[0] = C->n[0]; sizes_out[1] = C->n[1]; sizes_out[2] = 0; }
    plan->symbolic_ok = true;
    plan->m = S.m;
    plan->scratch = scratch;
    return SPWS_OK;
}

spws_status_t outer_numeric(spws_plan_s* plan, const Shapes& S, spws_tensor_t* C, void* scratch, size_t scratch_bytes) {
    const int64_t I = S.m, K = S.k, J = S.ncols, P = plan->outer_products;
    if (C->n[1] < plan->stats.nnz) return SPWS_OUTPUT_TOO_SMALL;
    if (plan->stats.nnz > 0 && (!C->crd[1] || !C->val)) return SPWS_INVALID_ARGUMENT;
    const OuterLayout L = make_outer_layout(plan, I, K, J, P);
    if (scratch_bytes < (plan->outer_dense ? L.dense_end : L.ism_end)) return SPWS_SCRATCH_TOO_SMALL;
    char* sc = static_cast<char*>(scratch);
    LaunchCtx c{};
    c.stream = plan->h->stream;
    c.sm_count = plan->h->sm_count;
    c.ctl = reinterpret_cast<DevCtl*>(sc + L.ctl);
    c.is_f64 = plan->is_f64;
    const size_t V = plan->is_f64 ? 8 : 4;
    i64* koff = reinterpret_cast<i64*>(sc + L.koff);
    i64* block_sums = reinterpret_cast<i64*>(sc + L.block_sums);
    mark_start(plan, 1);
    if (plan->outer_dense) {
        const size_t row_words = (size_t)((J + 31) / 32);
        CUDA_TRY(cudaMemsetAsync(sc + L.dbits, 0, 4 * (size_t)I * row_words, c.stream));
        CUDA_TRY(cudaMemsetAsync(sc + L.dvals, 0, V * (size_t)I * (size_t)J, c.stream));
        CUDA_TRY(launch_outer_dense(c, true, S.A, S.B, koff, P, I, J, reinterpret_cast<unsigned*>(sc + L.dbits), sc + L.dvals, nullptr,
                                    LL(C->pos[1]), C->crd[1], C->val));
        mark(plan, SPWS_T_NUM_DENSE_CTA);
    } else {
        bool first = true;
        i64* nnz_host = reinterpret_cast<i64*>(&plan->host_ctl->nnz);
        const int64_t cap = plan->opt.outer_cap > 0 ? plan->opt.outer_cap : (P > 0 ? P : 1);
        CUDA_TRY(launch_outer_ism(c, true, S.A, S.B, koff, P, cap, J, label_bits_of(I, J), reinterpret_cast<u64*>(sc + L.kA), sc + L.vA,
                                  reinterpret_cast<u64*>(sc + L.kB), sc + L.vB, reinterpret_cast<int*>(sc + L.head),
                                  reinterpret_cast<i64*>(sc + L.at), sc + L.sort_tmp, block_sums, &c.ctl->kept[0], nnz_host, &first));
        if (*nnz_host != plan->stats.nnz) return SPWS_BAD_SEQUENCE;     // operands differ from the symbolic pass's
        CUDA_TRY(launch_coo_out(c, reinterpret_cast<u64*>(sc + (first ? L.kA : L.kB)), sc + (first ? L.vA : L.vB), *nnz_host, J, C->crd[1], C->val));
        mark(plan, SPWS_T_NUM_ISM_GLOBAL);
    }
    plan->stats.launches_numeric = c.launches;
    return SPWS_OK;
}

// ---- higher-order scatters with coordinate-form output (kinds 3, 4, 5) -------------------------
struct HShapes {
    int form;                   // 0 SpTTM, 1 SpTTM-I, 2 SpMTTKRP
    Csf3Dev B;
    Csr C, D;
    int order;                  // of the output
    int64_t odims[3];
    u64 d1, d2;                 // label = (c_a * d1 + c_b) * d2 + c_c, or c_a * d2 + c_b
    int label_bits;
};

spws_status_t check_higher(const spws_plan_s* p, const spws_tensor_t* B, const spws_tensor_t* C, const spws_tensor_t* D, HShapes& H,
                           bool need_pointers) {
    if (!B || !C) return SPWS_INVALID_ARGUMENT;
    H.form = p->kind - 3;
    if ((H.form == 2) != (D != nullptr)) return SPWS_INVALID_ARGUMENT;
    if (B->order != 3 || C->order != 2 || (D && D->order != 2)) return SPWS_INVALID_ARGUMENT;
    for (int a = 0; a < 3; ++a)
        if (B->dims[a] < 0 || B->dims[a] > 0x7ffffff0ll || B->n[a] < 0) return SPWS_INVALID_ARGUMENT;
    if (B->n[0] > B->dims[0] || B->n[1] < B->n[0] || B->n[2] < B->n[1]) return SPWS_INVALID_ARGUMENT;
    if (C->dims[0] < 0 || C->dims[1] < 0 || C->dims[1] > 0x7ffffff0ll || C->n[1] < 0) return SPWS_INVALID_ARGUMENT;
    H.B = Csf3Dev{LL(B->pos[1]), LL(B->pos[2]), B->crd[0], B->crd[1], B->crd[2], B->val, (int)B->n[0], (int)B->n[1], B->n[2]};
    H.C = Csr{LL(C->pos[1]), C->crd[1], C->val, (int)C->dims[0], (int)C->dims[1]};
    H.D = Csr{};
    if (H.form == 0) {          // B(k,i,j), C(k,l) -> (i,j,l)
        if (C->dims[0] != B->dims[0]) return SPWS_DIM_MISMATCH;
        H.order = 3; H.odims[0] = B->dims[1]; H.odims[1] = B->dims[2]; H.odims[2] = C->dims[1];
    } else if (H.form == 1) {   // B(k,i,j), C(i,l) -> (k,j,l)
        if (C->dims[0] != B->dims[1]) return SPWS_DIM_MISMATCH;
        H.order = 3; H.odims[0] = B->dims[0]; H.odims[1] = B->dims[2]; H.odims[2] = C->dims[1];
    } else {                    // B(k,l,i), C(k,j), D(l,j) -> (i,j)
        if (C->dims[0] != B->dims[0] || D->dims[0] != B->dims[1] || D->dims[1] != C->dims[1]) return SPWS_DIM_MISMATCH;
        if (D->n[1] < 0) return SPWS_INVALID_ARGUMENT;
        H.D = Csr{LL(D->pos[1]), D->crd[1], D->val, (int)D->dims[0], (int)D->dims[1]};
        H.order = 2; H.odims[0] = B->dims[2]; H.odims[1] = C->dims[1]; H.odims[2] = 1;
    }
    // the label must fit 63 bits (one more is kept for the absent label)
    long double cells = 1.0L;
    for (int a = 0; a < H.order; ++a) cells *= (long double)(H.odims[a] > 0 ? H.odims[a] : 1);
    if (cells >= 4.0e18L) return SPWS_WORKSPACE_TOO_LARGE;
    H.d1 = H.order == 3 ? (u64)H.odims[1] : 1;
    H.d2 = (u64)H.odims[H.order - 1];
    u64 top = 1;
    for (int a = 0; a < H.order; ++a) top *= (u64)(H.odims[a] > 0 ? H.odims[a] : 1);
    H.label_bits = 1;
    while (H.label_bits < 63 && (top >> H.label_bits) != 0) ++H.label_bits;
    ++H.label_bits;             // the absent label's extra bit
    if (!need_pointers) return SPWS_OK;
    if (B->n[2] > 0 && (!H.B.pos1 || !H.B.pos2 || !H.B.crd0 || !H.B.crd1 || !H.B.crd2 || !H.B.val)) return SPWS_INVALID_ARGUMENT;
    if (C->dims[0] > 0 && !H.C.pos) return SPWS_INVALID_ARGUMENT;
    if (C->n[1] > 0 && (!H.C.crd || !H.C.val)) return SPWS_INVALID_ARGUMENT;
    if (D && ((D->dims[0] > 0 && !H.D.pos) || (D->n[1] > 0 && (!H.D.crd || !H.D.val)))) return SPWS_INVALID_ARGUMENT;
    return SPWS_OK;
}

struct HLayout {
    size_t ctl, fib_of, slice_of, cnt, eoff, block_sums, fixed_end, kA, kB, vA, vB, head, at, sort_tmp, end;
    int64_t N;
};

HLayout make_hlayout(const spws_plan_s* p, const HShapes& H, int64_t P) {
    HLayout L{};
    const size_t V = p->is_f64 ? 8 : 4;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align256(o + bytes); return at; };
    const int64_t cap = p->opt.outer_cap > 0 ? p->opt.outer_cap : P;
    L.N = P + (cap < P ? cap : 0);
    const int64_t longest = std::max<int64_t>(H.B.nnz, L.N);
    L.ctl = take(sizeof(DevCtl));
    L.fib_of = take(4 * (size_t)H.B.nnz);
    L.slice_of = take(4 * (size_t)H.B.n1);
    L.cnt = take(4 * (size_t)H.B.nnz);
    L.eoff = take(8 * ((size_t)H.B.nnz + 1));
    L.block_sums = take(8 * ((size_t)longest / 2048 + 2));
    L.fixed_end = o;
    L.kA = take(8 * (size_t)L.N);
    L.kB = take(8 * (size_t)L.N);
    L.vA = take(V * (size_t)L.N);
    L.vB = take(V * (size_t)L.N);
    L.head = take(4 * (size_t)L.N);
    L.at = take(8 * ((size_t)L.N + 1));
    L.sort_tmp = take(outer_sort_scratch_bytes(L.N));
    L.end = o;
    return L;
}

spws_status_t higher_count_products(spws_plan_s* p, const HShapes& H, int64_t* P) {
    LaunchCtx c{};
    c.stream = p->h->stream;
    c.sm_count = p->h->sm_count;
    u64* word = reinterpret_cast<u64*>(&p->host_ctl->products);
    *word = 0;
    CUDA_TRY(launch_higher_total(c, H.form, H.B, H.C, word));
    CUDA_TRY(cudaStreamSynchronize(c.stream));
    *P = (int64_t)*word;
    return SPWS_OK;
}

spws_status_t higher_workspace_size(spws_plan_s* plan, const spws_tensor_t* B, const spws_tensor_t* C, const spws_tensor_t* D, size_t* bytes) {
    HShapes H{};
    spws_status_t st = check_higher(plan, B, C, D, H, true);
    if (st != SPWS_OK) return st;
    int64_t P = 0;
    if ((st = higher_count_products(plan, H, &P)) != SPWS_OK) return st;
    *bytes = make_hlayout(plan, H, P).end;
    return SPWS_OK;
}

spws_status_t check_coo_output(const HShapes& H, const spws_tensor_t* Out) {
    if (!Out || Out->order != H.order) return SPWS_INVALID_ARGUMENT;
    for (int a = 0; a < H.order; ++a)
        if (Out->dims[a] != H.odims[a]) return SPWS_DIM_MISMATCH;
    return SPWS_OK;
}

spws_status_t higher_symbolic(spws_plan_s* plan, const spws_tensor_t* B, const spws_tensor_t* C, const spws_tensor_t* D, spws_tensor_t* Out,
                              void* scratch, size_t scratch_bytes, int64_t* sizes_out) {
    plan->symbolic_ok = false;
    HShapes H{};
    spws_status_t st = check_higher(plan, B, C, D, H, true);
    if (st != SPWS_OK) return st;
    if ((st = check_coo_output(H, Out)) != SPWS_OK) return st;
    if (!scratch || (reinterpret_cast<uintptr_t>(scratch) & 255)) return SPWS_INVALID_ARGUMENT;
    int64_t P = 0;
    if ((st = higher_count_products(plan, H, &P)) != SPWS_OK) return st;
    if (P > 0x7fff0000ll || H.B.nnz > 0x7fff0000ll) return SPWS_INTERNAL_OVERFLOW;       // ordinals and scans are 31-bit here
    const HLayout L = make_hlayout(plan, H, P);
    if (scratch_bytes < L.end) return SPWS_SCRATCH_TOO_SMALL;
    char* sc = static_cast<char*>(scratch);
    LaunchCtx c{};
    c.stream = plan->h->stream;
    c.sm_count = plan->h->sm_count;
    c.ctl = reinterpret_cast<DevCtl*>(sc + L.ctl);
    c.is_f64 = plan->is_f64;
    CUDA_TRY(cudaMemsetAsync(c.ctl, 0, sizeof(DevCtl), c.stream));
    mark_start(plan, 0);
    int* fib_of = reinterpret_cast<int*>(sc + L.fib_of);
    int* slice_of = reinterpret_cast<int*>(sc + L.slice_of);
    int* cnt = reinterpret_cast<int*>(sc + L.cnt);
    i64* eoff = reinterpret_cast<i64*>(sc + L.eoff);
    i64* block_sums = reinterpret_cast<i64*>(sc + L.block_sums);
    CUDA_TRY(launch_higher_setup(c, H.form, H.B, H.C, fib_of, slice_of, cnt));
    CUDA_TRY(launch_scan_counts(c, cnt, (int)H.B.nnz, eoff, block_sums, &c.ctl->products));
    mark(plan, SPWS_T_SYM_BOUNDS);
    bool first = true;
    i64* nnz_host = reinterpret_cast<i64*>(&plan->host_ctl->nnz);
    const int64_t cap = plan->opt.outer_cap > 0 ? plan->opt.outer_cap : (P > 0 ? P : 1);
    CUDA_TRY(launch_higher_ism(c, false, H.form, H.B, H.C, H.D, fib_of, slice_of, eoff, P, cap, H.d1, H.d2, H.label_bits,
                               reinterpret_cast<u64*>(sc + L.kA), nullptr, reinterpret_cast<u64*>(sc + L.kB), nullptr,
                               reinterpret_cast<int*>(sc + L.head), reinterpret_cast<i64*>(sc + L.at), sc + L.sort_tmp, block_sums,
                               &c.ctl->nnz, nnz_host, &first));
    const int64_t nnz = *nnz_host;
    mark(plan, SPWS_T_SYM_ISM_GLOBAL);
    CUDA_TRY(cudaMemcpyAsync(&plan->host_ctl->status, &c.ctl->status, sizeof(int), cudaMemcpyDeviceToHost, c.stream));
    CUDA_TRY(cudaStreamSynchronize(c.stream));
    plan->stats = spws_stats_t{};
    plan->stats.device_status = plan->host_ctl->status;
    if (plan->host_ctl->status != 0) return from_dev_status(plan->host_ctl->status);
    plan->stats.rows = H.B.nnz;
    plan->stats.products = P;
    plan->stats.nnz = nnz;
    plan->stats.rows_per_class[public_class(CLS_ISM_GLOBAL)] = H.B.nnz;
    plan->stats.products_per_class[public_class(CLS_ISM_GLOBAL)] = P;
    plan->stats.nnz_per_class[public_class(CLS_ISM_GLOBAL)] = nnz;
    plan->stats.launches_symbolic = c.launches;
    plan->outer_products = P;
    Out->n[0] = nnz; Out->n[1] = 0; Out->n[2] = 0;
    if (sizes_out) { sizes_out[0] = nnz; sizes_out[1] = 0; sizes_out[2] = 0; }
    plan->symbolic_ok = true;
    plan->m = H.B.nnz;
    plan->scratch = scratch;
    return SPWS_OK;
}

spws_status_t higher_numeric(spws_plan_s* plan, const spws_tensor_t* B, const spws_tensor_t* C, const spws_tensor_t* D, spws_tensor_t* Out,
                             void* scratch, size_t scratch_bytes) {
    if (!plan->symbolic_ok) return SPWS_BAD_SEQUENCE;
    HShapes H{};
    spws_status_t st = check_higher(plan, B, C, D, H, true);
    if (st != SPWS_OK) return st;
    if ((st = check_coo_output(H, Out)) != SPWS_OK) return st;
    if (scratch != plan->scratch || H.B.nnz != plan->m) return SPWS_BAD_SEQUENCE;
    const int64_t P = plan->outer_products, nnz = plan->stats.nnz;
    if (Out->n[0] < nnz) return SPWS_OUTPUT_TOO_SMALL;
    if (nnz > 0) {
        if (!Out->val) return SPWS_INVALID_ARGUMENT;
        for (int a = 0; a < H.order; ++a) if (!Out->crd[a]) return SPWS_INVALID_ARGUMENT;
    }
    const HLayout L = make_hlayout(plan, H, P);
    if (scratch_bytes < L.end) return SPWS_SCRATCH_TOO_SMALL;
    char* sc = static_cast<char*>(scratch);
    LaunchCtx c{};
    c.stream = plan->h->stream;
    c.sm_count = plan->h->sm_count;
    c.ctl = reinterpret_cast<DevCtl*>(sc + L.ctl);
    c.is_f64 = plan->is_f64;
    mark_start(plan, 1);
    bool first = true;
    i64* nnz_host = reinterpret_cast<i64*>(&plan->host_ctl->nnz);
    const int64_t cap = plan->opt.outer_cap > 0 ? plan->opt.outer_cap : (P > 0 ? P : 1);
    CUDA_TRY(launch_higher_ism(c, true, H.form, H.B, H.C, H.D, reinterpret_cast<int*>(sc + L.fib_of), reinterpret_cast<int*>(sc + L.slice_of),
                               reinterpret_cast<i64*>(sc + L.eoff), P, cap, H.d1, H.d2, H.label_bits, reinterpret_cast<u64*>(sc + L.kA),
                               sc + L.vA, reinterpret_cast<u64*>(sc + L.kB), sc + L.vB, reinterpret_cast<int*>(sc + L.head),
                               reinterpret_cast<i64*>(sc + L.at), sc + L.sort_tmp, reinterpret_cast<i64*>(sc + L.block_sums),
                               &c.ctl->kept[0], nnz_host, &first));
    if (*nnz_host != nnz) return SPWS_BAD_SEQUENCE;                 // operands differ from the symbolic pass's
    CUDA_TRY(launch_higher_unpack(c, H.order, reinterpret_cast<u64*>(sc + (first ? L.kA : L.kB)), sc + (first ? L.vA : L.vB), nnz, H.d1, H.d2,
                                  Out->crd[0], Out->crd[1], Out->crd[2], Out->val));
    mark(plan, SPWS_T_NUM_ISM_GLOBAL);
    plan->stats.launches_numeric = c.launches;
    return SPWS_OK;
}

}  // namespace

extern "C" {

spws_status_t spws_check_expression(const char* expr, const spws_format_t fmts[3], int* kind) {
    if (!expr || !fmts) return SPWS_INVALID_ARGUMENT;
    for (int f = 0; f < 3; ++f)
        if (fmts[f] != SPWS_CSR && fmts[f] != SPWS_CSF3 && fmts[f] != SPWS_COO) return SPWS_INVALID_ARGUMENT;
    const int k = classify_expression(expr, fmts, 3);
    if (k < 0) return SPWS_UNSUPPORTED_EXPRESSION;
    if (kind) *kind = k;
    return SPWS_OK;
}

spws_status_t spws_create(spws_handle_t* handle) {
    if (!handle) return SPWS_INVALID_ARGUMENT;
    spws_handle_s* h = new (std::nothrow) spws_handle_s;
    if (!h) return SPWS_INVALID_ARGUMENT;
    if (cudaGetDevice(&h->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device) != cudaSuccess) {
        cudaGetLastError();
        delete h;
        return SPWS_CUDA_ERROR;
    }
    *handle = h;
    return SPWS_OK;
}

spws_status_t spws_destroy(spws_handle_t handle) {
    if (!handle) return SPWS_INVALID_ARGUMENT;
    delete handle;
    return SPWS_OK;
}

spws_status_t spws_set_stream(spws_handle_t handle, void* cuda_stream) {
    if (!handle) return SPWS_INVALID_ARGUMENT;
    handle->stream = static_cast<cudaStream_t>(cuda_stream);
    return SPWS_OK;
}

static spws_status_t plan_create_n(spws_handle_t handle, const char* expr, const spws_format_t* fmts, int n_fmts,
                                   spws_dtype_t value_type, spws_policy_t policy, const spws_options_t* options,
                                   spws_plan_t* plan) {
    if (!handle || !expr || !fmts || !plan) return SPWS_INVALID_ARGUMENT;
    if (value_type != SPWS_F32 && value_type != SPWS_F64) return SPWS_INVALID_ARGUMENT;
    if (policy != SPWS_DENSE && policy != SPWS_SPARSE_ISM && policy != SPWS_AUTO && policy != SPWS_HASH) return SPWS_INVALID_ARGUMENT;
    for (int f = 0; f < n_fmts; ++f)
        if (fmts[f] != SPWS_CSR && fmts[f] != SPWS_CSF3 && fmts[f] != SPWS_COO) return SPWS_INVALID_ARGUMENT;
    const int kind = classify_expression(expr, fmts, n_fmts);
    if (kind < 0) return SPWS_UNSUPPORTED_EXPRESSION;
    if (kind >= 3 && policy == SPWS_DENSE) return SPWS_WORKSPACE_TOO_LARGE;      // no dense workspace of order three is offered
    spws_options_t o{};
    if (options) o = *options;
    const bool f64 = value_type == SPWS_F64;
    if (o.ism_warp_cap == 0) o.ism_warp_cap = 32;
    if (o.ism_cta_cap == 0) o.ism_cta_cap = 4096;
    if (o.dense_unit_outputs == 0) o.dense_unit_outputs = 4096;
    if (o.dense_max_span == 0) o.dense_max_span = 1 << 19;
    if (o.fallback_cap == 0) o.fallback_cap = 2048;
    if (o.dense_span_words_per_product == 0.0f) o.dense_span_words_per_product = 8.0f;
    if (o.validate != 0 && o.validate != 1) return SPWS_INVALID_ARGUMENT;
    if (o.ism_warp_cap < 1 || o.ism_warp_cap > 32) return SPWS_INVALID_ARGUMENT;
    if (!is_pow2(o.ism_cta_cap) || o.ism_cta_cap < 64 || o.ism_cta_cap > 4096) return SPWS_INVALID_ARGUMENT;
    if (!is_pow2(o.dense_unit_outputs) || o.dense_unit_outputs < 64 || o.dense_unit_outputs > 8192) return SPWS_INVALID_ARGUMENT;
    if (o.dense_max_span < 32 || o.dense_max_span > (1 << 19)) return SPWS_INVALID_ARGUMENT;
    if (!is_pow2(o.fallback_cap) || o.fallback_cap < 2 || o.fallback_cap > 2048) return SPWS_INVALID_ARGUMENT;
    if (!(o.dense_span_words_per_product > 0.0f)) return SPWS_INVALID_ARGUMENT;
    if (o.outer_cap < 0) return SPWS_INVALID_ARGUMENT;
    spws_plan_s* p = new (std::nothrow) spws_plan_s;
    if (!p) return SPWS_INVALID_ARGUMENT;
    p->h = handle;
    p->kind = kind;
    p->is_f64 = f64 ? 1 : 0;
    p->policy = (int)policy;
    p->opt = o;
    if (cudaMallocHost(reinterpret_cast<void**>(&p->host_ctl), sizeof(DevCtl)) != cudaSuccess) {
        cudaGetLastError();
        delete p;
        return SPWS_CUDA_ERROR;
    }
    memset(p->host_ctl, 0, sizeof(DevCtl));
    *plan = p;
    return SPWS_OK;
}

spws_status_t spws_plan_create(spws_handle_t handle, const char* expr, const spws_format_t fmts[3], spws_dtype_t value_type,
                               spws_policy_t policy, const spws_options_t* options, spws_plan_t* plan) {
    return plan_create_n(handle, expr, fmts, 3, value_type, policy, options, plan);
}

spws_status_t spws_plan_create3(spws_handle_t handle, const char* expr, const spws_format_t fmts[4], spws_dtype_t value_type,
                                spws_policy_t policy, const spws_options_t* options, spws_plan_t* plan) {
    return plan_create_n(handle, expr, fmts, 4, value_type, policy, options, plan);
}

spws_status_t spws_set_profiling(spws_plan_t plan, int enabled) {
    if (!plan) return SPWS_INVALID_ARGUMENT;
    if (enabled && !plan->ev[0]) {
        for (int g = 0; g < SPWS_T_COUNT; ++g) CUDA_TRY(cudaEventCreate(&plan->ev[g]));
        for (int g = 0; g < 3; ++g) CUDA_TRY(cudaEventCreate(&plan->ev_start[g]));
    }
    plan->profiling = enabled != 0;
    return SPWS_OK;
}

spws_status_t spws_get_timings(spws_plan_t plan, float* ms, int n) {
    if (!plan || !ms || n < SPWS_T_COUNT) return SPWS_INVALID_ARGUMENT;
    for (int g = 0; g < SPWS_T_COUNT; ++g) ms[g] = 0.0f;
    if (!plan->ev[0]) return SPWS_BAD_SEQUENCE;
    CUDA_TRY(cudaStreamSynchronize(plan->h->stream));
    for (int pass = 0; pass < 3; ++pass) {
        if (!plan->ev_pass[pass]) continue;
        cudaEvent_t prev = plan->ev_start[pass];
        const int g0 = PASS_GROUPS[pass], g1 = PASS_GROUPS[pass + 1];
        for (int g = g0; g < g1; ++g) {
            if (!plan->ev_ran[g]) continue;
            CUDA_TRY(cudaEventElapsedTime(&ms[g], prev, plan->ev[g]));
            prev = plan->ev[g];
        }
    }
    return SPWS_OK;
}

spws_status_t spws_plan_destroy(spws_plan_t plan) {
    if (!plan) return SPWS_INVALID_ARGUMENT;
    if (plan->ev[0]) {
        for (int g = 0; g < SPWS_T_COUNT; ++g) cudaEventDestroy(plan->ev[g]);
        for (int g = 0; g < 3; ++g) cudaEventDestroy(plan->ev_start[g]);
    }
    if (plan->host_ctl) cudaFreeHost(plan->host_ctl);
    delete plan;
    return SPWS_OK;
}

spws_status_t spws_workspace_size(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B, size_t* bytes) {
    if (!plan || !bytes) return SPWS_INVALID_ARGUMENT;
    if (plan->kind == 5) return SPWS_INVALID_ARGUMENT;           // three operands: spws_workspace_size3
    if (plan->kind >= 3) return higher_workspace_size(plan, A, B, nullptr, bytes);
    Shapes S{};
    spws_status_t st = check_operands(plan, A, B, S, plan->kind != 2);   // pointers may still be unset when sizing
    if (st != SPWS_OK) return st;
    if (plan->kind == 2) {                      // sized by the number of products, counted on the device
        int64_t P = 0;
        if ((st = outer_count_products(plan, S, &P)) != SPWS_OK) return st;
        const OuterLayout OL = make_outer_layout(plan, S.m, S.k, S.ncols, P);
        const size_t dense_ok = (double)S.m * (double)S.ncols <= 2.0e9 ? OL.dense_end : 0;     // a dense workspace beyond 2^31 cells is never offered
        *bytes = (plan->policy == SPWS_SPARSE_ISM || plan->policy == SPWS_HASH) ? OL.ism_end
                 : plan->policy == SPWS_DENSE ? OL.dense_end
                 : std::max(OL.ism_end, ((double)S.m * (double)S.ncols <= 134217728.0 || (double)P * 16.0 >= (double)S.m * (double)S.ncols) ? dense_ok : (size_t)0);
        return SPWS_OK;
    }
    const Layout L = make_layout(plan, S.m, S.ncols, S.n_i, S.nnzB, S.k, S.nnzA);
    *bytes = L.fixed_end + rest_reserve(plan, S.m, S.ncols);
    return SPWS_OK;
}

spws_status_t spws_workspace_size_exact(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B, void* scratch,
                                        size_t scratch_bytes, size_t* bytes, int64_t* row_products) {
    if (!plan || !bytes) return SPWS_INVALID_ARGUMENT;
    if (plan->kind >= 2) return spws_workspace_size(plan, A, B, bytes);      // already sized from the product count
    Shapes S{};
    spws_status_t st = check_operands(plan, A, B, S, scratch != nullptr);
    if (st != SPWS_OK) return st;
    const Layout L = make_layout(plan, S.m, S.ncols, S.n_i, S.nnzB, S.k, S.nnzA);
    if (!scratch) {                             // first step of the protocol: what this call itself needs
        *bytes = L.fixed_end;
        return SPWS_OK;
    }
    if (reinterpret_cast<uintptr_t>(scratch) & 255) return SPWS_INVALID_ARGUMENT;
    if (scratch_bytes < L.fixed_end) return SPWS_SCRATCH_TOO_SMALL;
    plan->symbolic_ok = false;                  // the tables of an earlier symbolic pass are overwritten
    char* sc = static_cast<char*>(scratch);
    LaunchCtx c = make_ctx(plan, sc, scratch_bytes, L);
    c.prm.bm_arena_words = ~0ull >> 3;          // reserve without a limit: only the total is wanted
    CUDA_TRY(cudaMemsetAsync(c.ctl, 0, sizeof(DevCtl), c.stream));
    CUDA_TRY(launch_row_bounds(c, S.A, S.B, S.nnzA));
    CUDA_TRY(launch_bin_rows(c, (int)S.m));
    if (row_products && S.m > 0)
        CUDA_TRY(cudaMemcpyAsync(row_products, c.tab.ub, 8 * (size_t)S.m, cudaMemcpyDeviceToDevice, c.stream));
    CUDA_TRY(cudaMemcpyAsync(plan->host_ctl, c.ctl, sizeof(DevCtl), cudaMemcpyDeviceToHost, c.stream));
    CUDA_TRY(cudaStreamSynchronize(c.stream));
    const DevCtl& hc = *plan->host_ctl;
    if (hc.status != 0 && hc.status != DEV_SCRATCH_TOO_SMALL) return from_dev_status(hc.status);
    size_t need = L.fixed_end + align256((size_t)hc.bm_words_used * 4);
    const int64_t n_global = hc.class_count[CLS_ISM_GLOBAL];
    if (n_global > 0) {                         // numeric slots of the global-memory ISM, sized for its largest row
        int64_t elems = hc.max_ub_global < S.ncols ? hc.max_ub_global : S.ncols;
        elems = (elems + 63) & ~63ll;
        const size_t comp = 4 + (plan->is_f64 ? 8 : 4);
        const size_t slot = align256(2 * (size_t)elems * comp);
        need += slot * global_ism_slots(plan, slot, n_global);
    }
    *bytes = need;
    return SPWS_OK;
}

spws_status_t spws_symbolic(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B, spws_tensor_t* C,
                            void* scratch, size_t scratch_bytes, int64_t* sizes_out) {
    if (!plan) return SPWS_INVALID_ARGUMENT;
    if (plan->kind == 5) return SPWS_INVALID_ARGUMENT;
    if (plan->kind >= 3) return higher_symbolic(plan, A, B, nullptr, C, scratch, scratch_bytes, sizes_out);
    plan->symbolic_ok = false;
    Shapes S{};
    spws_status_t st = check_operands(plan, A, B, S);
    if (st != SPWS_OK) return st;
    if ((st = check_output_dims(plan, A, B, C)) != SPWS_OK) return st;
    if (!scratch || (reinterpret_cast<uintptr_t>(scratch) & 255)) return SPWS_INVALID_ARGUMENT;
    if (plan->kind == 2) return outer_symbolic(plan, S, C, scratch, scratch_bytes, sizes_out);
    const Layout L = make_layout(plan, S.m, S.ncols, S.n_i, S.nnzB, S.k, S.nnzA);
    if (scratch_bytes < L.fixed_end) return SPWS_SCRATCH_TOO_SMALL;
    char* sc = static_cast<char*>(scratch);
    LaunchCtx c = make_ctx(plan, sc, scratch_bytes, L);
    cudaStream_t stream = c.stream;

    CUDA_TRY(cudaMemsetAsync(c.ctl, 0, sizeof(DevCtl), stream));
    if (plan->opt.validate) {
        CUDA_TRY(launch_validate(c, S.A, S.B, S.nnzA, S.nnzB));
        CUDA_TRY(cudaMemcpyAsync(plan->host_ctl, c.ctl, sizeof(DevCtl), cudaMemcpyDeviceToHost, stream));
        CUDA_TRY(cudaStreamSynchronize(stream));
        if (plan->host_ctl->status != 0) return from_dev_status(plan->host_ctl->status);
    }
    // a1: upper bounds + classes; a2: binning
    mark_start(plan, 0);
    CUDA_TRY(launch_row_bounds(c, S.A, S.B, S.nnzA));
    CUDA_TRY(launch_bw_build(c, S.B));
    mark(plan, SPWS_T_SYM_BOUNDS);
    CUDA_TRY(launch_bin_rows(c, (int)S.m));
    mark(plan, SPWS_T_SYM_BIN);
    // the class sizes come back now, so that only the workspaces that have rows are launched, with
    // grids sized for them (a launch for an empty class costs as much as a small class's work)
    int* hcount = plan->host_ctl->class_count;
    CUDA_TRY(cudaMemcpyAsync(hcount, c.ctl->class_count, sizeof(int) * NCLASS, cudaMemcpyDeviceToHost, stream));
    CUDA_TRY(cudaMemcpyAsync(&plan->host_ctl->max_ub_smem, &c.ctl->max_ub_smem, sizeof(i64), cudaMemcpyDeviceToHost, stream));
    CUDA_TRY(cudaStreamSynchronize(stream));
    plan->max_ub_smem = plan->host_ctl->max_ub_smem;
    c.max_ub_smem = plan->max_ub_smem;
    // a3: exact count per row through the workspace of its class
    i64* rowptr = (plan->kind == 0) ? LL(C->pos[1]) : reinterpret_cast<i64*>(sc + L.rowptr_raw);
    if (S.m > 0) {
        for (int cls = CLS_ISM_REG8; cls <= CLS_ISM_REG; ++cls)
            if (hcount[cls] > 0) {
                CUDA_TRY(launch_ism_reg(c, false, cls, hcount[cls], S.A, S.B, rowptr, nullptr, nullptr));
                mark(plan, SPWS_T_SYM_ISM_REG);
            }
        // under `auto` the rows of the shared-memory insert-sort-merge classes are counted through a
        // hash set of their columns: the count needs no order
        const bool count_by_hash = plan->policy == SPWS_AUTO;
        if (hcount[CLS_ISM_SMEM_S] > 0) {
            if (count_by_hash) CUDA_TRY(launch_hash(c, false, CLS_ISM_SMEM_S, hcount[CLS_ISM_SMEM_S], S.A, S.B, rowptr, nullptr, nullptr));
            else CUDA_TRY(launch_ism_smem(c, false, CLS_ISM_SMEM_S, hcount[CLS_ISM_SMEM_S], S.A, S.B, rowptr, nullptr, nullptr));
            mark(plan, SPWS_T_SYM_ISM_SMEM_S);
        }
        if (hcount[CLS_ISM_SMEM] > 0) {
            if (count_by_hash) CUDA_TRY(launch_hash(c, false, CLS_ISM_SMEM, hcount[CLS_ISM_SMEM], S.A, S.B, rowptr, nullptr, nullptr));
            else CUDA_TRY(launch_ism_smem(c, false, CLS_ISM_SMEM, hcount[CLS_ISM_SMEM], S.A, S.B, rowptr, nullptr, nullptr));
            mark(plan, SPWS_T_SYM_ISM_SMEM);
        }
        if (hcount[CLS_DENSE_WARP] > 0) {
            CUDA_TRY(launch_dense_sym_warp(c, S.A, S.B));
            mark(plan, SPWS_T_SYM_DENSE_WARP);
        }
        if (hcount[CLS_DENSE_HUB] + hcount[CLS_DENSE_CTA] > 0) {
            CUDA_TRY(launch_dense_sym_cta(c, S.A, S.B));
            mark(plan, SPWS_T_SYM_DENSE_CTA);
        }
        if (hcount[CLS_ISM_GLOBAL] > 0) {
            CUDA_TRY(launch_ism_global(c, false, hcount[CLS_ISM_GLOBAL], S.A, S.B, rowptr, nullptr, nullptr));
            mark(plan, SPWS_T_SYM_ISM_GLOBAL);
        }
        for (int cls = CLS_HASH_S; cls <= CLS_HASH; ++cls)
            if (hcount[cls] > 0) {
                CUDA_TRY(launch_hash(c, false, cls, hcount[cls], S.A, S.B, rowptr, nullptr, nullptr));
                mark(plan, SPWS_T_SYM_HASH);
            }
    }
    // a4: exclusive scan into the row pointer
    if (plan->kind == 1) {
        // with C's fibre and slice levels rebuilt from the fibres that produced an output
        CUDA_TRY(launch_ttm_scan_compact(c, (int)S.n_i, (int)S.m, LL(A->pos[1]), A->crd[0], A->crd[1], rowptr,
                                         reinterpret_cast<i64*>(sc + L.fpos), reinterpret_cast<int*>(sc + L.sflags),
                                         reinterpret_cast<i64*>(sc + L.spos), reinterpret_cast<i64*>(sc + L.block_sums), &c.ctl->nnz,
                                         LL(C->pos[0]), C->crd[0], LL(C->pos[1]), C->crd[1], LL(C->pos[2])));
    } else {
        CUDA_TRY(launch_scan_counts(c, c.tab.cnt, (int)S.m, rowptr, reinterpret_cast<i64*>(sc + L.block_sums), &c.ctl->nnz));
    }
    if (hcount[CLS_DENSE_WARP] + hcount[CLS_DENSE_HUB] + hcount[CLS_DENSE_CTA] > 0) CUDA_TRY(launch_dense_rebin(c, (int)S.m, rowptr));
    CUDA_TRY(launch_class_nnz(c, (int)S.m));
    mark(plan, SPWS_T_SYM_SCAN);
    CUDA_TRY(cudaMemcpyAsync(plan->host_ctl, c.ctl, sizeof(DevCtl), cudaMemcpyDeviceToHost, stream));
    CUDA_TRY(cudaStreamSynchronize(stream));
    const DevCtl& hc = *plan->host_ctl;
    plan->stats = spws_stats_t{};
    plan->stats.device_status = hc.status;
    if (hc.status != 0) return from_dev_status(hc.status);
    plan->stats.rows = S.m;
    plan->stats.products = hc.products;
    plan->stats.nnz = hc.nnz;
    plan->stats.max_row_products = hc.max_ub;
    for (int k = 0; k < NCLASS; ++k) {
        plan->bin_rows[k] = hc.class_count[k];
        plan->stats.rows_per_class[public_class(k)] += hc.class_count[k];
        plan->stats.products_per_class[public_class(k)] += hc.class_products[k];
        plan->stats.nnz_per_class[public_class(k)] += hc.class_nnz[k];
    }
    plan->stats.dense_units = hc.n_units;
    plan->stats.dense_warp_rows = hc.n_warp_rows;
    plan->stats.dense_warp_products = hc.dense_warp_products;
    plan->stats.dense_warp_nnz = hc.dense_warp_nnz;
    plan->stats.bitmap_bytes = (int64_t)hc.bm_words_used * 4;
    plan->max_span_words = hc.max_span_words;
    plan->max_warp_cnt = hc.max_warp_cnt;
    plan->stats.launches_symbolic = c.launches;
    if (plan->kind == 0) {
        C->n[0] = C->dims[0];
        C->n[1] = hc.nnz;
        C->n[2] = 0;
    } else {
        C->n[0] = hc.kept[0];
        C->n[1] = hc.kept[1];
        C->n[2] = hc.nnz;
    }
    if (sizes_out) { sizes_out[0] = C->n[0]; sizes_out[1] = C->n[1]; sizes_out[2] = C->n[2]; }
    plan->symbolic_ok = true;
    plan->m = S.m;
    plan->scratch = scratch;
    return SPWS_OK;
}

spws_status_t spws_numeric(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B, spws_tensor_t* C,
                           void* scratch, size_t scratch_bytes) {
    if (!plan) return SPWS_INVALID_ARGUMENT;
    if (plan->kind == 5) return SPWS_INVALID_ARGUMENT;
    if (plan->kind >= 3) return higher_numeric(plan, A, B, nullptr, C, scratch, scratch_bytes);
    if (!plan->symbolic_ok) return SPWS_BAD_SEQUENCE;
    Shapes S{};
    spws_status_t st = check_operands(plan, A, B, S);
    if (st != SPWS_OK) return st;
    if ((st = check_output_dims(plan, A, B, C)) != SPWS_OK) return st;
    if (scratch != plan->scratch || S.m != plan->m) return SPWS_BAD_SEQUENCE;
    if (plan->kind == 2) return outer_numeric(plan, S, C, scratch, scratch_bytes);
    const int last = plan->kind == 0 ? 1 : 2;
    if (C->n[last] < plan->stats.nnz) return SPWS_OUTPUT_TOO_SMALL;
    if (plan->stats.nnz > 0 && (!C->crd[last] || !C->val)) return SPWS_INVALID_ARGUMENT;
    const Layout L = make_layout(plan, S.m, S.ncols, S.n_i, S.nnzB, S.k, S.nnzA);
    if (scratch_bytes < L.fixed_end) return SPWS_SCRATCH_TOO_SMALL;
    char* sc = static_cast<char*>(scratch);
    LaunchCtx c = make_ctx(plan, sc, scratch_bytes, L);
    const i64* rowptr = (plan->kind == 0) ? LL(C->pos[1]) : reinterpret_cast<const i64*>(sc + L.rowptr_raw);
    CUDA_TRY(cudaMemsetAsync(c.ctl->work_counter, 0, sizeof(c.ctl->work_counter), c.stream));
    mark_start(plan, 1);
    c.max_ub_smem = plan->max_ub_smem;
    const spws_stats_t& s = plan->stats;
    int* crd = C->crd[last];
    const int64_t* bins = plan->bin_rows;
    for (int cls : {(int)CLS_COPY8, (int)CLS_ISM_REG8, (int)CLS_ISM_REG16, (int)CLS_ISM_REG})
        if (bins[cls] > 0) {
            CUDA_TRY(launch_ism_reg(c, true, cls, (int)bins[cls], S.A, S.B, rowptr, crd, C->val));
            mark(plan, SPWS_T_NUM_ISM_REG);
        }
    if (bins[CLS_ISM_SMEM_S] > 0) {
        CUDA_TRY(launch_ism_smem(c, true, CLS_ISM_SMEM_S, (int)bins[CLS_ISM_SMEM_S], S.A, S.B, rowptr, crd, C->val));
        mark(plan, SPWS_T_NUM_ISM_SMEM_S);
    }
    if (bins[CLS_ISM_SMEM] > 0) {
        CUDA_TRY(launch_ism_smem(c, true, CLS_ISM_SMEM, (int)bins[CLS_ISM_SMEM], S.A, S.B, rowptr, crd, C->val));
        mark(plan, SPWS_T_NUM_ISM_SMEM);
    }
    if (s.dense_warp_rows > 0) {
        CUDA_TRY(launch_dense_num_warp(c, (int)s.dense_warp_rows, plan->max_span_words, plan->max_warp_cnt, S.A, S.B, rowptr, crd, C->val));
        mark(plan, SPWS_T_NUM_DENSE_WARP);
    }
    if (s.dense_units > 0) {
        CUDA_TRY(launch_dense_num_cta(c, 0, (int)s.dense_units, plan->max_span_words, s.products, S.A, S.B, rowptr, crd, C->val));
        mark(plan, SPWS_T_NUM_DENSE_EMIT);
        CUDA_TRY(launch_dense_num_cta(c, 1, (int)s.dense_units, plan->max_span_words, s.products, S.A, S.B, rowptr, crd, C->val));
        mark(plan, SPWS_T_NUM_DENSE_CTA);
    }
    if (bins[CLS_ISM_GLOBAL] > 0) {
        CUDA_TRY(launch_ism_global(c, true, (int)bins[CLS_ISM_GLOBAL], S.A, S.B, rowptr, crd, C->val));
        mark(plan, SPWS_T_NUM_ISM_GLOBAL);
    }
    for (int cls = CLS_HASH_S; cls <= CLS_HASH; ++cls)
        if (bins[cls] > 0) {
            CUDA_TRY(launch_hash(c, true, cls, (int)bins[cls], S.A, S.B, rowptr, crd, C->val));
            mark(plan, SPWS_T_NUM_HASH);
        }
    plan->stats.launches_numeric = c.launches;
    return SPWS_OK;
}

spws_status_t spws_gather_ceiling(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B, const spws_tensor_t* C,
                                  void* scratch, size_t scratch_bytes, uint64_t* index_sum, double* value_sum) {
    if (!plan || !index_sum || !value_sum) return SPWS_INVALID_ARGUMENT;
    if (plan->kind >= 2) return SPWS_UNSUPPORTED_EXPRESSION;    // the first-order dense kernels run for the row-wise forms only
    if (!plan->symbolic_ok) return SPWS_BAD_SEQUENCE;
    Shapes S{};
    spws_status_t st = check_operands(plan, A, B, S);
    if (st != SPWS_OK) return st;
    if ((st = check_output_dims(plan, A, B, C)) != SPWS_OK) return st;
    if (scratch != plan->scratch || S.m != plan->m) return SPWS_BAD_SEQUENCE;
    const Layout L = make_layout(plan, S.m, S.ncols, S.n_i, S.nnzB, S.k, S.nnzA);
    if (scratch_bytes < L.fixed_end) return SPWS_SCRATCH_TOO_SMALL;
    char* sc = static_cast<char*>(scratch);
    LaunchCtx c = make_ctx(plan, sc, scratch_bytes, L);
    const i64* rowptr = (plan->kind == 0) ? LL(C->pos[1]) : reinterpret_cast<const i64*>(sc + L.rowptr_raw);
    CUDA_TRY(cudaMemsetAsync(c.ctl->work_counter + CEIL_SLOT, 0, sizeof(int) * NCLASS, c.stream));
    CUDA_TRY(cudaMemsetAsync(index_sum, 0, sizeof(uint64_t), c.stream));
    CUDA_TRY(cudaMemsetAsync(value_sum, 0, sizeof(double), c.stream));
    mark_start(plan, 2);
    const spws_stats_t& s = plan->stats;
    u64* ci = reinterpret_cast<u64*>(index_sum);
    if (s.dense_warp_rows > 0) {
        CUDA_TRY(launch_dense_num_warp(c, (int)s.dense_warp_rows, plan->max_span_words, plan->max_warp_cnt, S.A, S.B, rowptr, nullptr, nullptr, ci, value_sum));
        mark(plan, SPWS_T_CEIL_DENSE_WARP);
    }
    if (s.dense_units > 0) {
        CUDA_TRY(launch_dense_num_cta(c, 1, (int)s.dense_units, plan->max_span_words, s.products, S.A, S.B, rowptr, nullptr, nullptr, ci, value_sum));
        mark(plan, SPWS_T_CEIL_DENSE_CTA);
    }
    return SPWS_OK;
}

spws_status_t spws_get_stats(spws_plan_t plan, spws_stats_t* stats) {
    if (!plan || !stats) return SPWS_INVALID_ARGUMENT;
    if (!plan->symbolic_ok) return SPWS_BAD_SEQUENCE;
    DevCtl* ctl = reinterpret_cast<DevCtl*>(plan->scratch);
    CUDA_TRY(cudaMemcpyAsync(&plan->host_ctl->status, &ctl->status, sizeof(int), cudaMemcpyDeviceToHost, plan->h->stream));
    CUDA_TRY(cudaStreamSynchronize(plan->h->stream));
    plan->stats.device_status = plan->host_ctl->status;
    *stats = plan->stats;
    return from_dev_status(plan->host_ctl->status);
}

spws_status_t spws_workspace_size3(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B, const spws_tensor_t* D, size_t* bytes) {
    if (!plan || !bytes || plan->kind != 5) return SPWS_INVALID_ARGUMENT;
    return higher_workspace_size(plan, A, B, D, bytes);
}

spws_status_t spws_symbolic3(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B, const spws_tensor_t* D, spws_tensor_t* C,
                             void* scratch, size_t scratch_bytes, int64_t* sizes_out) {
    if (!plan || plan->kind != 5) return SPWS_INVALID_ARGUMENT;
    return higher_symbolic(plan, A, B, D, C, scratch, scratch_bytes, sizes_out);
}

spws_status_t spws_numeric3(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B, const spws_tensor_t* D, spws_tensor_t* C,
                            void* scratch, size_t scratch_bytes) {
    if (!plan || plan->kind != 5) return SPWS_INVALID_ARGUMENT;
    return higher_numeric(plan, A, B, D, C, scratch, scratch_bytes);
}

spws_status_t spws_execute_host(spws_plan_t plan, const spws_tensor_t* A, const spws_tensor_t* B, spws_tensor_t* C,
                                void* arena, size_t arena_bytes, size_t* arena_needed) {
    if (!plan || !A || !B || !C || !arena) return SPWS_INVALID_ARGUMENT;
    if (plan->kind >= 3) return SPWS_UNSUPPORTED_EXPRESSION;     // host entry: the CSR / CSF result forms only
    if (reinterpret_cast<uintptr_t>(arena) & 255) return SPWS_INVALID_ARGUMENT;
    Shapes S{};
    spws_status_t st = check_operands(plan, A, B, S);
    if (st != SPWS_OK) return st;
    cudaStream_t stream = plan->h->stream;
    const size_t V = plan->is_f64 ? 8 : 4;
    char* base = static_cast<char*>(arena);
    size_t o = 0;
    bool fits = true;
    auto carve = [&](size_t bytes) -> char* {
        char* at = base + o;
        o = align256(o + bytes);
        if (o > arena_bytes) fits = false;
        return at;
    };
    // device images of the operands
    spws_tensor_t dA = *A, dB = *B, dC = *C;
    const int lastA = plan->kind == 0 ? 1 : 2;
    const bool same = (plan->kind != 1) && A->pos[1] == B->pos[1] && A->crd[1] == B->crd[1] && A->val == B->val;
    struct Copy { void* dst; const void* src; size_t bytes; };
    std::vector<Copy> h2d;
    auto stage = [&](const void* src, size_t bytes) -> void* {
        char* d = carve(bytes);
        h2d.push_back(Copy{d, src, bytes});
        return d;
    };
    if (plan->kind != 1) {
        dA.pos[1] = (int64_t*)stage(A->pos[1], 8 * ((size_t)A->dims[0] + 1));
        dA.crd[1] = (int32_t*)stage(A->crd[1], 4 * (size_t)S.nnzA);
    } else {
        dA.pos[0] = (int64_t*)stage(A->pos[0], 16);
        dA.crd[0] = (int32_t*)stage(A->crd[0], 4 * (size_t)A->n[0]);
        dA.pos[1] = (int64_t*)stage(A->pos[1], 8 * ((size_t)A->n[0] + 1));
        dA.crd[1] = (int32_t*)stage(A->crd[1], 4 * (size_t)A->n[1]);
        dA.pos[2] = (int64_t*)stage(A->pos[2], 8 * ((size_t)A->n[1] + 1));
        dA.crd[2] = (int32_t*)stage(A->crd[2], 4 * (size_t)S.nnzA);
    }
    dA.val = stage(A->val, V * (size_t)S.nnzA);
    if (same) {
        dB.pos[1] = dA.pos[1]; dB.crd[1] = dA.crd[1]; dB.val = dA.val;
    } else {
        dB.pos[1] = (int64_t*)stage(B->pos[1], 8 * ((size_t)B->dims[0] + 1));
        dB.crd[1] = (int32_t*)stage(B->crd[1], 4 * (size_t)S.nnzB);
        dB.val = stage(B->val, V * (size_t)S.nnzB);
    }
    (void)lastA;
    if (plan->kind != 1) {
        dC.pos[1] = (int64_t*)carve(8 * ((size_t)S.m + 1));
    } else {
        dC.pos[0] = (int64_t*)carve(16);
        dC.crd[0] = (int32_t*)carve(4 * (size_t)A->n[0]);
        dC.pos[1] = (int64_t*)carve(8 * ((size_t)A->n[0] + 1));
        dC.crd[1] = (int32_t*)carve(4 * (size_t)A->n[1]);
        dC.pos[2] = (int64_t*)carve(8 * ((size_t)A->n[1] + 1));
    }
    if (!fits) {
        if (arena_needed) *arena_needed = o;      // lower bound: scratch and C's entries are not counted yet
        return SPWS_SCRATCH_TOO_SMALL;
    }
    for (const Copy& cp : h2d)
        if (cp.bytes) CUDA_TRY(cudaMemcpyAsync(cp.dst, cp.src, cp.bytes, cudaMemcpyHostToDevice, stream));
    size_t ws_bytes = 0;                          // the outer-product form sizes its workspace from the device copies
    if ((st = spws_workspace_size(plan, plan->kind == 2 ? &dA : A, plan->kind == 2 ? &dB : B, &ws_bytes)) != SPWS_OK) return st;
    char* scratch = carve(ws_bytes);
    if (!fits) {
        if (arena_needed) *arena_needed = o;      // lower bound: C's entries are not counted yet
        return SPWS_SCRATCH_TOO_SMALL;
    }
    int64_t cap[3] = {C->n[0], C->n[1], C->n[2]};
    int64_t sizes[3];
    if ((st = spws_symbolic(plan, &dA, &dB, &dC, scratch, ws_bytes, sizes)) != SPWS_OK) return st;
    const int last = plan->kind == 1 ? 2 : 1;
    const size_t nnz = (size_t)sizes[last];
    dC.crd[last] = (int32_t*)carve(4 * nnz);
    dC.val = carve(V * nnz);
    if (arena_needed) *arena_needed = o;
    C->n[0] = sizes[0]; C->n[1] = sizes[1]; C->n[2] = sizes[2];
    if (!fits) return SPWS_SCRATCH_TOO_SMALL;
    if ((int64_t)nnz > cap[last]) return SPWS_OUTPUT_TOO_SMALL;
    if (plan->kind == 1 && (sizes[0] > cap[0] || sizes[1] > cap[1])) return SPWS_OUTPUT_TOO_SMALL;
    if ((st = spws_numeric(plan, &dA, &dB, &dC, scratch, ws_bytes)) != SPWS_OK) return st;
    if (plan->kind != 1) {
        CUDA_TRY(cudaMemcpyAsync(C->pos[1], dC.pos[1], 8 * ((size_t)S.m + 1), cudaMemcpyDeviceToHost, stream));
    } else {
        CUDA_TRY(cudaMemcpyAsync(C->pos[0], dC.pos[0], 16, cudaMemcpyDeviceToHost, stream));
        if (sizes[0]) CUDA_TRY(cudaMemcpyAsync(C->crd[0], dC.crd[0], 4 * (size_t)sizes[0], cudaMemcpyDeviceToHost, stream));
        CUDA_TRY(cudaMemcpyAsync(C->pos[1], dC.pos[1], 8 * ((size_t)sizes[0] + 1), cudaMemcpyDeviceToHost, stream));
        if (sizes[1]) CUDA_TRY(cudaMemcpyAsync(C->crd[1], dC.crd[1], 4 * (size_t)sizes[1], cudaMemcpyDeviceToHost, stream));
        CUDA_TRY(cudaMemcpyAsync(C->pos[2], dC.pos[2], 8 * ((size_t)sizes[1] + 1), cudaMemcpyDeviceToHost, stream));
    }
    if (nnz) {
        CUDA_TRY(cudaMemcpyAsync(C->crd[last], dC.crd[last], 4 * nnz, cudaMemcpyDeviceToHost, stream));
        CUDA_TRY(cudaMemcpyAsync(C->val, dC.val, V * nnz, cudaMemcpyDeviceToHost, stream));
    }
    spws_stats_t stats;
    return spws_get_stats(plan, &stats);
}

const char* spws_status_string(spws_status_t status) {
    switch (status) {
        case SPWS_OK: return "ok";
        case SPWS_INVALID_ARGUMENT: return "invalid argument";
        case SPWS_UNSUPPORTED_EXPRESSION: return "unsupported expression";
        case SPWS_DIM_MISMATCH: return "dimension mismatch";
        case SPWS_NONCANONICAL_INPUT: return "non-canonical input";
        case SPWS_SCRATCH_TOO_SMALL: return "scratch too small";
        case SPWS_WORKSPACE_TOO_LARGE: return "dense workspace too large";
        case SPWS_CUDA_ERROR: return "CUDA error";
        case SPWS_INTERNAL_OVERFLOW: return "internal overflow";
        case SPWS_OUTPUT_TOO_SMALL: return "output too small";
        case SPWS_BAD_SEQUENCE: return "bad call sequence";
    }
    return "unknown status";
}

}  // extern "C"
