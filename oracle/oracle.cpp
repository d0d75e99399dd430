// TEST INFRASTRUCTURE ONLY -- the CPU oracle.  Nothing in the product path may call it.
//
// Plain, slow, sequential-per-row definitions of what the sparse-workspace path computes,
// written from the paper's statement of the problem.  It shares no code with the CUDA path.
//
//   oracle_spgemm   : row-wise SpGEMM  C(i,j) = sum_k A(i,k) * B(k,j), all CSR.  One ordered
//                     map per output row: a product either lands on an existing coordinate
//                     (deduplicate = sum) or is inserted as a new one (Sec. 1, Fig. 1; Sec. 4.3);
//                     loop order i -> k -> j (Sec. 2.2); coordinates of a row come out sorted and
//                     unique (Sec. 4.2).  An entry whose sum happens to be 0.0 is kept: Compress
//                     copies every stored component (Fig. 8, Compress part).
//   oracle_ttm      : C(i,j,l) = sum_k A(i,j,k) * B(k,l), A and C in CSF (three compressed
//                     levels), B CSR.  The outer loops i, j are shared by producer and consumer
//                     (common iteration hoisting, Sec. 6.2) so each (i,j) fibre gets a first-order
//                     map over l; fibres (and slices) with no output are not materialised, as
//                     Compress only creates coordinates that exist (Fig. 8, Compress part).
//   oracle_ism_rowwise / oracle_ism_outer :
//                     Algorithm 1 taken step by step (Allocate; Insert; on full: Sort, Merge,
//                     Insert again; tail Sort+Merge; Compress) with the Coord policy of Sec. 5.2
//                     (append, no reduction on insert, lexicographic sort at flush) and an
//                     out-of-place two-way Merge that reduces equal coordinates (Sec. 4.3).  The
//                     row-wise form uses a first-order workspace per row; the outer form follows
//                     the loop order k -> i -> j of the paper's running example (Sec. 2.1) with a
//                     second-order workspace and the COO -> CSR Compress.  Reading of the
//                     "Insert / if full / Insert again" protocol: an Insert into an accumulation
//                     array that has no free slot stores nothing and raises `full`; the same
//                     component is inserted again after the flush.
//
// Values: `val` is the double-precision sum taken in loop order (multiply, then add; built with
// -ffp-contract=off); `val_ref` accumulates the same products in long double and rounds once;
// `abs` is sum |a*b| (the scale of the forward error bound of a reordered sum).
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <map>
#include <thread>
#include <utility>
#include <vector>

namespace {

struct Cell {
    double sum = 0.0;
    long double ref = 0.0L;
    double abs = 0.0;
};

struct Result {
    // CSR result (spgemm) or CSF level 2 (ttm): pos over rows / fibres.
    std::vector<int64_t> pos;
    std::vector<int32_t> crd;
    std::vector<double> val, val_ref, abs;
    std::vector<int64_t> products;   // intermediate products per row / input fibre
    // CSF upper levels (ttm only)
    std::vector<int64_t> pos0, pos1;
    std::vector<int32_t> crd0, crd1;
};

struct Csr {
    const int64_t* pos;
    const int32_t* crd;
    const double* val;
};

// One output row: the ordered-map workspace.
void row_into_map(const Csr& A, const Csr& B, int64_t i, std::map<int32_t, Cell>& ws, int64_t& products) {
    for (int64_t p = A.pos[i]; p < A.pos[i + 1]; ++p) {
        const int32_t k = A.crd[p];
        const double a = A.val[p];
        for (int64_t q = B.pos[k]; q < B.pos[k + 1]; ++q) {
            const double prod = a * B.val[q];
            Cell& c = ws[B.crd[q]];          // inserts a zero cell when the coordinate is new
            c.sum += prod;
            c.ref += static_cast<long double>(a) * static_cast<long double>(B.val[q]);
            c.abs += std::fabs(prod);
            ++products;
        }
    }
}

struct RowBlockOut {
    std::vector<int64_t> cnt, products;
    std::vector<int32_t> crd;
    std::vector<double> val, val_ref, abs;
};

void run_rows(const Csr& A, const Csr& B, const int64_t* rows, int64_t r0, int64_t r1, RowBlockOut& out) {
    std::map<int32_t, Cell> ws;
    for (int64_t r = r0; r < r1; ++r) {
        const int64_t i = rows ? rows[r] : r;
        ws.clear();
        int64_t products = 0;
        row_into_map(A, B, i, ws, products);
        out.cnt.push_back(static_cast<int64_t>(ws.size()));
        out.products.push_back(products);
        for (const auto& kv : ws) {
            out.crd.push_back(kv.first);
            out.val.push_back(kv.second.sum);
            out.val_ref.push_back(static_cast<double>(kv.second.ref));
            out.abs.push_back(kv.second.abs);
        }
    }
}

template <class T>
void append(std::vector<T>& dst, const std::vector<T>& src) {
    dst.insert(dst.end(), src.begin(), src.end());
}

// ---- Algorithm 1 pieces (Coord policy) -------------------------------------------------

struct Component {
    int32_t crd[2];
    double val;
};

inline bool crd_less(const Component& a, const Component& b) {
    return a.crd[0] < b.crd[0] || (a.crd[0] == b.crd[0] && a.crd[1] < b.crd[1]);
}
inline bool crd_equal(const Component& a, const Component& b) {
    return a.crd[0] == b.crd[0] && a.crd[1] == b.crd[1];
}

struct AccArray {
    std::vector<Component> slot;
    size_t cap;
    bool full = false;
    explicit AccArray(size_t c) : cap(c) { slot.reserve(c); }
    bool empty() const { return slot.empty(); }
};

// Insert: append when a slot is free, otherwise store nothing and raise `full`.
void Insert(const Component& c, AccArray& acc) {
    if (acc.slot.size() < acc.cap) {
        acc.slot.push_back(c);
        acc.full = false;
    } else {
        acc.full = true;
    }
}

// Sort: lexicographic order of the coordinates; equal coordinates are then adjacent and are
// reduced here (the Coord policy does not reduce on insert).
void Sort(AccArray& acc) {
    std::stable_sort(acc.slot.begin(), acc.slot.end(), crd_less);
    std::vector<Component> uniq;
    for (const Component& c : acc.slot) {
        if (!uniq.empty() && crd_equal(uniq.back(), c)) uniq.back().val += c.val;
        else uniq.push_back(c);
    }
    acc.slot.swap(uniq);
}

// Merge: out-of-place two-way merge of the sorted accumulation array into the sorted all
// array, reducing equal coordinates; clears the accumulation array.
void Merge(AccArray& acc, std::vector<Component>& all) {
    std::vector<Component> out;
    out.reserve(all.size() + acc.slot.size());
    size_t x = 0, y = 0;
    while (x < all.size() && y < acc.slot.size()) {
        if (crd_equal(all[x], acc.slot[y])) {
            Component c = all[x++];
            c.val += acc.slot[y++].val;
            out.push_back(c);
        } else if (crd_less(all[x], acc.slot[y])) {
            out.push_back(all[x++]);
        } else {
            out.push_back(acc.slot[y++]);
        }
    }
    while (x < all.size()) out.push_back(all[x++]);
    while (y < acc.slot.size()) out.push_back(acc.slot[y++]);
    all.swap(out);
    acc.slot.clear();
    acc.full = false;
}

void insert_with_flush(const Component& c, AccArray& acc, std::vector<Component>& all) {
    Insert(c, acc);
    if (acc.full) {
        Sort(acc);
        Merge(acc, all);
        Insert(c, acc);
    }
}

}  // namespace

extern "C" {

// rows == nullptr: all m rows; otherwise the n_sel listed rows, in the order given.
void* oracle_spgemm(int64_t m, const int64_t* Apos, const int32_t* Acrd, const double* Aval,
                    const int64_t* Bpos, const int32_t* Bcrd, const double* Bval,
                    const int64_t* rows, int64_t n_sel, int nthreads) {
    const Csr A{Apos, Acrd, Aval}, B{Bpos, Bcrd, Bval};
    const int64_t n = rows ? n_sel : m;
    if (nthreads < 1) nthreads = 1;
    if (nthreads > n) nthreads = n > 0 ? static_cast<int>(n) : 1;
    std::vector<RowBlockOut> parts(nthreads);
    // contiguous blocks balanced on A's nonzero count (rows are independent)
    std::vector<int64_t> cut(nthreads + 1, n);
    cut[0] = 0;
    {
        int64_t total = 0;
        for (int64_t r = 0; r < n; ++r) { const int64_t i = rows ? rows[r] : r; total += Apos[i + 1] - Apos[i] + 1; }
        int64_t acc = 0; int t = 1;
        for (int64_t r = 0; r < n && t < nthreads; ++r) {
            const int64_t i = rows ? rows[r] : r;
            acc += Apos[i + 1] - Apos[i] + 1;
            while (t < nthreads && acc >= total * t / nthreads) cut[t++] = r + 1;
        }
    }
    if (nthreads == 1) {
        run_rows(A, B, rows, 0, n, parts[0]);
    } else {
        std::vector<std::thread> th;
        for (int t = 0; t < nthreads; ++t)
            th.emplace_back([&, t] { run_rows(A, B, rows, cut[t], cut[t + 1], parts[t]); });
        for (auto& t : th) t.join();
    }
    Result* R = new Result;
    R->pos.push_back(0);
    for (auto& p : parts) {
        for (int64_t c : p.cnt) R->pos.push_back(R->pos.back() + c);
        append(R->products, p.products);
        append(R->crd, p.crd);
        append(R->val, p.val);
        append(R->val_ref, p.val_ref);
        append(R->abs, p.abs);
    }
    return R;
}

void* oracle_ttm(int64_t n_i, const int32_t* Acrd0, const int64_t* Apos1, const int32_t* Acrd1,
                 const int64_t* Apos2, const int32_t* Acrd2, const double* Aval,
                 const int64_t* Bpos, const int32_t* Bcrd, const double* Bval) {
    Result* R = new Result;
    R->pos.push_back(0);
    R->pos1.push_back(0);
    const Csr fibres{Apos2, Acrd2, Aval}, B{Bpos, Bcrd, Bval};
    std::map<int32_t, Cell> ws;
    for (int64_t s = 0; s < n_i; ++s) {                       // level 0: stored i coordinates
        int64_t kept_j = 0;
        for (int64_t f = Apos1[s]; f < Apos1[s + 1]; ++f) {   // level 1: the (i,j) fibres
            ws.clear();
            int64_t products = 0;
            row_into_map(fibres, B, f, ws, products);         // level 2 workspace over l
            R->products.push_back(products);
            if (ws.empty()) continue;
            ++kept_j;
            R->crd1.push_back(Acrd1[f]);
            for (const auto& kv : ws) {
                R->crd.push_back(kv.first);
                R->val.push_back(kv.second.sum);
                R->val_ref.push_back(static_cast<double>(kv.second.ref));
                R->abs.push_back(kv.second.abs);
            }
            R->pos.push_back(static_cast<int64_t>(R->crd.size()));
        }
        if (kept_j > 0) {
            R->crd0.push_back(Acrd0[s]);
            R->pos1.push_back(R->pos1.back() + kept_j);
        }
    }
    R->pos0 = {0, static_cast<int64_t>(R->crd0.size())};
    return R;
}

// Algorithm 1, first-order workspace per output row (key = j), capacity `cap` >= 1.
void* oracle_ism_rowwise(int64_t m, const int64_t* Apos, const int32_t* Acrd, const double* Aval,
                         const int64_t* Bpos, const int32_t* Bcrd, const double* Bval, int64_t cap) {
    Result* R = new Result;
    R->pos.push_back(0);
    for (int64_t i = 0; i < m; ++i) {
        AccArray acc(static_cast<size_t>(cap));               // Allocate
        std::vector<Component> all;
        for (int64_t p = Apos[i]; p < Apos[i + 1]; ++p) {
            const int32_t k = Acrd[p];
            for (int64_t q = Bpos[k]; q < Bpos[k + 1]; ++q) {
                Component c;
                c.crd[0] = 0;
                c.crd[1] = Bcrd[q];
                c.val = Aval[p] * Bval[q];
                insert_with_flush(c, acc, all);
            }
        }
        if (!acc.empty()) { Sort(acc); Merge(acc, all); }
        for (const Component& c : all) { R->crd.push_back(c.crd[1]); R->val.push_back(c.val); }  // Compress
        R->pos.push_back(static_cast<int64_t>(R->crd.size()));
    }
    R->val_ref = R->val;
    return R;
}

// Algorithm 1, second-order workspace, loop order k -> i -> j.  At holds A by columns, i.e.
// the CSR arrays of A transposed (K rows): row k lists the i with A(i,k) != 0.
void* oracle_ism_outer(int64_t m, int64_t K, const int64_t* Atpos, const int32_t* Atcrd, const double* Atval,
                       const int64_t* Bpos, const int32_t* Bcrd, const double* Bval, int64_t cap) {
    AccArray acc(static_cast<size_t>(cap));
    std::vector<Component> all;
    for (int64_t k = 0; k < K; ++k) {
        for (int64_t p = Atpos[k]; p < Atpos[k + 1]; ++p) {
            Component c;
            c.crd[0] = Atcrd[p];
            for (int64_t q = Bpos[k]; q < Bpos[k + 1]; ++q) {
                c.crd[1] = Bcrd[q];
                c.val = Atval[p] * Bval[q];
                insert_with_flush(c, acc, all);
            }
        }
    }
    if (!acc.empty()) { Sort(acc); Merge(acc, all); }
    // Compress: COO -> CSR.  Count the components of each row segment, then prefix-sum.
    Result* R = new Result;
    R->pos.assign(static_cast<size_t>(m) + 1, 0);
    size_t w = 0;
    while (w < all.size()) {
        const int32_t i = all[w].crd[0];
        size_t end = w + 1;
        while (end < all.size() && all[end].crd[0] == i) ++end;
        R->pos[static_cast<size_t>(i) + 1] = static_cast<int64_t>(end - w);
        w = end;
    }
    for (int64_t r = 1; r <= m; ++r) R->pos[r] += R->pos[r - 1];
    for (const Component& c : all) { R->crd.push_back(c.crd[1]); R->val.push_back(c.val); }
    R->val_ref = R->val;
    return R;
}

int64_t oracle_size(void* h, int what) {
    Result* R = static_cast<Result*>(h);
    switch (what) {
        case 0: return static_cast<int64_t>(R->pos.size());
        case 1: return static_cast<int64_t>(R->crd.size());
        case 2: return static_cast<int64_t>(R->products.size());
        case 3: return static_cast<int64_t>(R->crd0.size());
        case 4: return static_cast<int64_t>(R->crd1.size());
        case 5: return static_cast<int64_t>(R->pos1.size());
        case 6: return static_cast<int64_t>(R->abs.size());
    }
    return -1;
}

void oracle_copy(void* h, int what, void* dst) {
    Result* R = static_cast<Result*>(h);
    auto cp = [dst](const auto& v) { if (!v.empty()) std::memcpy(dst, v.data(), v.size() * sizeof(v[0])); };
    switch (what) {
        case 0: cp(R->pos); break;
        case 1: cp(R->crd); break;
        case 2: cp(R->val); break;
        case 3: cp(R->val_ref); break;
        case 4: cp(R->abs); break;
        case 5: cp(R->products); break;
        case 6: cp(R->pos0); break;
        case 7: cp(R->crd0); break;
        case 8: cp(R->pos1); break;
        case 9: cp(R->crd1); break;
    }
}

void oracle_free(void* h) { delete static_cast<Result*>(h); }

int oracle_hardware_threads() { return static_cast<int>(std::thread::hardware_concurrency()); }

}  // extern "C"
