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
//                     the insert-sort-merge workspace of Algorithm 1 under the coordinate-sort
//                     policy of Sec. 5.2 (append without reduction; sort and reduce when the
//                     bounded buffer is emptied; union with the sorted store of everything seen
//                     so far, Sec. 4.3), as a second, independent route to the same result.  The
//                     row-wise form gives every output row a first-order workspace; the outer form
//                     feeds one second-order workspace in the order k -> i -> j of Sec. 2.1 and
//                     converts the sorted coordinate list to CSR.  Reading of the algorithm's
//                     "insert, and if that found the buffer full, flush and insert again": an
//                     insert into a buffer without a free slot stores nothing; the same entry goes
//                     in after the flush.
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

// ---- Algorithm 1 with the coordinate-sort policy ---------------------------------------
//
// Written from the contract of Algorithm 1 (Sec. 4.2-4.3) and of the Coord policy (Sec. 5.2):
// a bounded buffer of pending (coordinate, value) entries in arrival order, and one store of
// settled entries that is always sorted by coordinate and free of duplicates.  An entry is
// offered to the buffer; when the buffer has no room it is emptied first -- its entries are
// put in coordinate order, equal coordinates are summed (this policy reduces at sort time, not
// at insert time), and the result is united with the settled store, again summing equal
// coordinates -- and the same entry is offered again.  What is still pending at the end is
// emptied the same way.  The settled store is then the whole result in storage order.

struct Entry {
    int32_t i, j;      // coordinate; first-order use keeps i = 0
    double v;
};

inline bool before(const Entry& a, const Entry& b) { return a.i != b.i ? a.i < b.i : a.j < b.j; }
inline bool same_place(const Entry& a, const Entry& b) { return a.i == b.i && a.j == b.j; }

class BoundedWorkspace {
public:
    explicit BoundedWorkspace(int64_t capacity) : capacity_(static_cast<size_t>(capacity)) { pending_.reserve(capacity_); }

    void feed(const Entry& e) {
        if (pending_.size() == capacity_) settle();      // no room: nothing is stored, empty the buffer ...
        pending_.push_back(e);                           // ... and take the same entry afterwards
    }

    // Moves everything pending into the settled store.
    void settle() {
        if (pending_.empty()) return;
        // order by coordinate, keeping arrival order among equals, then sum runs of equals
        std::stable_sort(pending_.begin(), pending_.end(), before);
        size_t kept = 0;
        for (size_t x = 0; x < pending_.size(); ++x) {
            if (kept > 0 && same_place(pending_[kept - 1], pending_[x])) pending_[kept - 1].v += pending_[x].v;
            else pending_[kept++] = pending_[x];
        }
        pending_.resize(kept);
        // union of two duplicate-free sorted sequences into a fresh one; a coordinate present in
        // both becomes settled value + pending value
        std::vector<Entry> joined(settled_.size() + pending_.size());
        std::merge(settled_.begin(), settled_.end(), pending_.begin(), pending_.end(), joined.begin(), before);
        kept = 0;
        for (size_t x = 0; x < joined.size(); ++x) {
            if (kept > 0 && same_place(joined[kept - 1], joined[x])) joined[kept - 1].v += joined[x].v;
            else joined[kept++] = joined[x];
        }
        joined.resize(kept);
        settled_.swap(joined);
        pending_.clear();
    }

    const std::vector<Entry>& settled() const { return settled_; }

private:
    size_t capacity_;
    std::vector<Entry> pending_, settled_;
};

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

// Algorithm 1, one first-order workspace per output row (coordinate = j), capacity `cap` >= 1.
void* oracle_ism_rowwise(int64_t m, const int64_t* Apos, const int32_t* Acrd, const double* Aval,
                         const int64_t* Bpos, const int32_t* Bcrd, const double* Bval, int64_t cap) {
    Result* R = new Result;
    R->pos.push_back(0);
    for (int64_t i = 0; i < m; ++i) {
        BoundedWorkspace ws(cap);
        for (int64_t p = Apos[i]; p < Apos[i + 1]; ++p) {
            const int32_t k = Acrd[p];
            for (int64_t q = Bpos[k]; q < Bpos[k + 1]; ++q) ws.feed(Entry{0, Bcrd[q], Aval[p] * Bval[q]});
        }
        ws.settle();
        for (const Entry& e : ws.settled()) { R->crd.push_back(e.j); R->val.push_back(e.v); }
        R->pos.push_back(static_cast<int64_t>(R->crd.size()));
    }
    R->val_ref = R->val;
    return R;
}

// Algorithm 1 with ONE second-order workspace (coordinate = (i, j)) for the whole product, fed
// in the outer-product order of Sec. 2.1: for each k, every stored A(i,k) times every stored
// B(k,j).  At holds A by columns, i.e. the CSR arrays of A transposed (K rows): row k lists the
// i with A(i,k) != 0.  The settled store is the result in coordinate (COO) form; turning it into
// CSR needs the number of entries of each row, prefix-summed.
void* oracle_ism_outer(int64_t m, int64_t K, const int64_t* Atpos, const int32_t* Atcrd, const double* Atval,
                       const int64_t* Bpos, const int32_t* Bcrd, const double* Bval, int64_t cap) {
    BoundedWorkspace ws(cap);
    for (int64_t k = 0; k < K; ++k)
        for (int64_t p = Atpos[k]; p < Atpos[k + 1]; ++p)
            for (int64_t q = Bpos[k]; q < Bpos[k + 1]; ++q) ws.feed(Entry{Atcrd[p], Bcrd[q], Atval[p] * Bval[q]});
    ws.settle();
    Result* R = new Result;
    std::vector<int64_t> per_row(static_cast<size_t>(m), 0);
    for (const Entry& e : ws.settled()) {
        ++per_row[static_cast<size_t>(e.i)];
        R->crd.push_back(e.j);
        R->val.push_back(e.v);
    }
    R->pos.assign(1, 0);
    for (int64_t r = 0; r < m; ++r) R->pos.push_back(R->pos.back() + per_row[static_cast<size_t>(r)]);
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
