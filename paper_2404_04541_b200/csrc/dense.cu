// Dense workspace: an occupancy bitmap along the last index plus a value array (Gustavson's
// workspace, Table 2: the flag marks positions that already hold a component, so a product
// deduplicates on insertion; position = coordinate, so the workspace is bucket-sorted; the
// flagged positions are copied out in order = boolean indexing).
//
// The bitmap covers the row's exact column span [jmin, jmax] and lives in shared memory.  The
// value array is NOT indexed by column but by the RANK of the column among the row's set bits
// (rank = prefix popcount), so it holds only as many entries as the row has outputs and is
// already in output order:
//   symbolic : gather the column indices of the row's products, set bits; cnt = popcount; the
//              bitmap is saved to the arena in scratch so the numeric pass need not rebuild it.
//   numeric  : reload the bitmap, prefix-sum its words, then acc[rank(j)] += a*b for every
//              product; acc is copied straight to the row's value segment and the set bits give
//              the column indices.
// Two granularities:
//   warp per row : bitmap <= 1024 words, <= 256 outputs.  A warp walks the A entries one at a
//              time with its lanes across the B row, so no two lanes ever hit the same slot and
//              the accumulator needs no atomics; sums are in loop order.
//   CTA units    : any span up to 2^19 columns.  A unit is a row, or an equal share of the A
//              entries of a row with very many products, so hub rows spread over many CTAs.
//              The first `unit_outputs` outputs of the row accumulate in shared memory
//              (atomics combine the CTA's warps), the rest in the row's value segment.  The
//              coordinates of these rows are written by a kernel of their own, which also clears
//              the value segments that several units add into.
#include "common.cuh"

namespace spws {

constexpr int DW_THREADS = 256;            // warp-per-row kernels: 8 warps per CTA
constexpr int DW_WARPS = DW_THREADS / 32;
constexpr int DC_THREADS = 256;            // symbolic CTA kernel
constexpr int DC_WARPS = DC_THREADS / 32;
constexpr int DN_THREADS = 512;            // numeric CTA kernel
constexpr int DN_WARPS = DN_THREADS / 32;

// A warp-route row whose bitmap is mostly empty words saves only the non-empty ones; bm_off then
// carries a flag and the number of saved words above the slot offset.
constexpr i64 BM_COMPACT = 1ll << 62;
constexpr int BM_NZW_SHIFT = 44;
constexpr i64 BM_OFF_MASK = (1ll << BM_NZW_SHIFT) - 1;

// A dense row's slot in the arena: nw bitmap words, then for every chunk of 32 words the rank of
// the chunk's first bit (an exclusive prefix of the chunk popcounts).
__device__ __forceinline__ int chunks_of(int nw) { return (nw + 31) >> 5; }

// lanes per A entry: the smallest power of two >= the mean B-row segment length
__device__ __forceinline__ int pick_group_size(i64 ub, i64 entries, int parts) {
    const float avg = (float)ub / fmaxf(1.0f, (float)entries * (float)parts);
    int gs = 32;
    while (gs > 1 && (float)(gs >> 1) >= avg) gs >>= 1;
    return gs;
}

// ---------------------------------------------------------------------------------------
// symbolic, warp per row
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(DW_THREADS) dense_sym_warp_kernel(DevCtl* __restrict__ ctl, Csr A, Csr B, RowTables tab) {
    __shared__ unsigned s_bm[DW_WARPS][DENSE_WARP_BM_WORDS];
    // bit w of the summary = bitmap word w is non-empty, so the copy-out walks only those words
    __shared__ unsigned s_sum[DW_WARPS][DENSE_WARP_BM_WORDS / 32];
    // descriptors of 32 A entries: (start of the B row << 16) | its length (a warp row has <= 4096 products)
    __shared__ __align__(16) u64 s_desc[DW_WARPS][32];
    if (ctl->status != 0) return;
    int off, n;
    class_range(ctl, CLS_DENSE_WARP, off, n);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned* bm = s_bm[warp];
    unsigned* sum = s_sum[warp];
    u64* desc = s_desc[warp];
    for (int w = lane; w < DENSE_WARP_BM_WORDS; w += 32) bm[w] = 0;     // every row leaves its bitmap clear
    sum[lane] = 0;
    __syncwarp();
    for (;;) {
        int r = 0;
        if (lane == 0) r = atomicAdd(&ctl->work_counter[CLS_DENSE_WARP], 1);
        r = __shfl_sync(0xffffffffu, r, 0);
        if (r >= n) break;
        const int row = tab.perm[off + r];
        const int base = tab.jmin[row];
        const int nw = (tab.jmax[row] - base) / 32 + 1;
        const unsigned span = (unsigned)nw * 32u;
        const i64 ps = A.pos[row], pe = A.pos[row + 1];
        const int gs = pick_group_size(tab.ub[row], pe - ps, 1);
        // the lane that sets a bit first counts the output; the lane that touches a word first
        // counts the word and flags it in the summary
        int cnt = 0, nzw = 0;
        auto mark = [&](unsigned rel) {
            if (rel < span) {
                const unsigned w = rel >> 5, bit = 1u << (rel & 31);
                const unsigned old = atomicOr(&bm[w], bit);
                if (!(old & bit)) {
                    ++cnt;
                    if (old == 0u) { ++nzw; atomicOr(&sum[w >> 5], 1u << (w & 31)); }
                }
            }
        };
        if (gs == 32) {
            // descriptors of 32 A entries at a time (one per lane, passed through shared memory), then
            // the first 32 elements of four B rows are loaded before any is consumed, to keep loads
            // in flight
            for (i64 p0 = ps; p0 < pe; p0 += 32) {
                u64 mine = 0;
                if (p0 + lane < pe) {
                    const int k = __ldg(A.crd + p0 + lane);
                    if ((unsigned)k < (unsigned)B.nrows) {
                        const i64 qs = __ldg(B.pos + k);
                        mine = ((u64)qs << 16) | (u64)(__ldg(B.pos + k + 1) - qs);
                    }
                }
                __syncwarp();
                desc[lane] = mine;
                __syncwarp();
                const int nE = (int)min((i64)32, pe - p0);
                for (int e = 0; e < nE; e += 4) {
                    const ulonglong2 d01 = *reinterpret_cast<const ulonglong2*>(desc + e);
                    const ulonglong2 d23 = *reinterpret_cast<const ulonglong2*>(desc + e + 2);
                    const u64 d[4] = {d01.x, d01.y, d23.x, d23.y};
                    i64 qs[4];
                    int len[4];
                    unsigned rel[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        qs[x] = (i64)(d[x] >> 16);
                        len[x] = (int)(d[x] & 0xffffu);                  // 0 past the last entry
                        rel[x] = (lane < len[x]) ? (unsigned)(__ldg(B.crd + qs[x] + lane) - base) : 0xffffffffu;
                    }
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        mark(rel[x]);
                        for (int t = lane + 32; t < len[x]; t += 32) mark((unsigned)(__ldg(B.crd + qs[x] + t) - base));
                    }
                }
            }
        } else {
            const int g = lane / gs, gl = lane % gs, ng = 32 / gs;
            for (i64 p = ps + g; p < pe; p += ng) {
                const int k = __ldg(A.crd + p);
                if ((unsigned)k >= (unsigned)B.nrows) continue;
                const i64 qs = __ldg(B.pos + k);
                const int len = (int)(__ldg(B.pos + k + 1) - qs);
                const int* __restrict__ ck = B.crd + qs;
                for (int t = gl; t < len; t += gs) mark((unsigned)(__ldg(ck + t) - base));
            }
        }
        for (int d = 16; d > 0; d >>= 1) {
            cnt += __shfl_xor_sync(0xffffffffu, cnt, d);
            nzw += __shfl_xor_sync(0xffffffffu, nzw, d);
        }
        __syncwarp();
        const i64 slot = tab.bm_off[row];
        unsigned* out = tab.bm_arena + slot;
        if (cnt <= DENSE_WARP_ACC && 2 * nzw <= nw + chunks_of(nw)) {
            // compact form for the warp numeric kernel: only the non-empty words, as (bits, word
            // index) in column order; lane l owns the words its summary word flags
            uint2* out2 = reinterpret_cast<uint2*>(out);
            unsigned s = sum[lane];
            sum[lane] = 0;
            const int c = __popc(s);
            int at = warp_incl_scan(c) - c;
            while (s) {
                const int w = (lane << 5) + __ffs(s) - 1;
                s &= s - 1;
                out2[at++] = make_uint2(bm[w], (unsigned)w);
                bm[w] = 0;
            }
            if (lane == 0) tab.bm_off[row] = slot | ((i64)nzw << BM_NZW_SHIFT) | BM_COMPACT;
        } else {
            // full form: every word, then the rank at every 32-word chunk start
            sum[lane] = 0;
            int carry = 0;
            for (int w0 = 0; w0 < nw; w0 += 32) {
                const int w = w0 + lane;
                const unsigned word = (w < nw) ? bm[w] : 0u;
                if (w < nw) { out[w] = word; bm[w] = 0; }
                int c = __popc(word);
                for (int d = 16; d > 0; d >>= 1) c += __shfl_xor_sync(0xffffffffu, c, d);
                if (lane == 0) out[nw + (w0 >> 5)] = (unsigned)carry;
                carry += c;
            }
        }
        if (lane == 0) tab.cnt[row] = cnt;
        __syncwarp();
    }
}

// ---------------------------------------------------------------------------------------
// symbolic, CTA per row (hub rows first: classes HUB and CTA are adjacent in perm)
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(DC_THREADS) dense_sym_cta_kernel(DevCtl* __restrict__ ctl, int smem_words, Csr A, Csr B, RowTables tab,
                                                                   const uint2* __restrict__ bw) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned* bm = reinterpret_cast<unsigned*>(smem_raw);                 // smem_words
    int* chunk = reinterpret_cast<int*>(bm + smem_words);                  // smem_words / 32
    __shared__ int s_next;
    __shared__ int ws[33];
    if (ctl->status != 0) return;
    int off, n_hub, o6, n_cta;
    class_range(ctl, CLS_DENSE_HUB, off, n_hub);
    class_range(ctl, CLS_DENSE_CTA, o6, n_cta);
    const int n = n_hub + n_cta;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (;;) {
        __syncthreads();
        if (tid == 0) s_next = atomicAdd(&ctl->work_counter[CLS_DENSE_CTA], 1);
        __syncthreads();
        const int r = s_next;
        if (r >= n) break;
        const int row = tab.perm[off + r];
        const int base = tab.jmin[row];
        const int nw = min((tab.jmax[row] - base) / 32 + 1, smem_words);
        const unsigned span = (unsigned)nw * 32u;
        const unsigned base_w = (unsigned)base >> 5;                     // base is a multiple of 32
        const i64 ps = A.pos[row], pe = A.pos[row + 1];
        for (int w = tid; w < nw; w += DC_THREADS) bm[w] = 0;
        __syncthreads();
        const int gs = pick_group_size(tab.ub[row], pe - ps, 1);
        const int g = tid / gs, gl = tid % gs, ng = DC_THREADS / gs;
        for (i64 p = ps + g; p < pe; p += ng) {
            const int k = __ldg(A.crd + p);
            if ((unsigned)k >= (unsigned)B.nrows) continue;
            const i64 qs = __ldg(B.pos + k);
            const int len = (int)(__ldg(B.pos + k + 1) - qs);
            if (bw && len >= BW_MIN_LEN) {
                // a long B row with a word list: one atomic per (word, bits) pair, and the lanes
                // of a warp hold distinct words
                const int np = (int)__ldg(&bw[qs].x);
                if (np > 0) {
                    const uint2* __restrict__ pk = bw + qs + 1;
                    int t = gl;
                    for (; t + 3 * gs < np; t += 4 * gs) {
                        const uint2 e0 = __ldg(pk + t), e1 = __ldg(pk + t + gs), e2 = __ldg(pk + t + 2 * gs), e3 = __ldg(pk + t + 3 * gs);
                        const unsigned w0 = e0.x - base_w, w1 = e1.x - base_w, w2 = e2.x - base_w, w3 = e3.x - base_w;
                        if (w0 < (unsigned)nw) atomicOr(&bm[w0], e0.y);
                        if (w1 < (unsigned)nw) atomicOr(&bm[w1], e1.y);
                        if (w2 < (unsigned)nw) atomicOr(&bm[w2], e2.y);
                        if (w3 < (unsigned)nw) atomicOr(&bm[w3], e3.y);
                    }
                    for (; t < np; t += gs) {
                        const uint2 e0 = __ldg(pk + t);
                        const unsigned w0 = e0.x - base_w;
                        if (w0 < (unsigned)nw) atomicOr(&bm[w0], e0.y);
                    }
                    continue;
                }
            }
            const int* __restrict__ ck = B.crd + qs;
            int t = gl;
            for (; t + 3 * gs < len; t += 4 * gs) {     // four loads in flight per lane
                const unsigned r0 = (unsigned)(__ldg(ck + t) - base);
                const unsigned r1 = (unsigned)(__ldg(ck + t + gs) - base);
                const unsigned r2 = (unsigned)(__ldg(ck + t + 2 * gs) - base);
                const unsigned r3 = (unsigned)(__ldg(ck + t + 3 * gs) - base);
                if (r0 < span) atomicOr(&bm[r0 >> 5], 1u << (r0 & 31));
                if (r1 < span) atomicOr(&bm[r1 >> 5], 1u << (r1 & 31));
                if (r2 < span) atomicOr(&bm[r2 >> 5], 1u << (r2 & 31));
                if (r3 < span) atomicOr(&bm[r3 >> 5], 1u << (r3 & 31));
            }
            for (; t < len; t += gs) {
                const unsigned r0 = (unsigned)(__ldg(ck + t) - base);
                if (r0 < span) atomicOr(&bm[r0 >> 5], 1u << (r0 & 31));
            }
        }
        __syncthreads();
        // save the bitmap, then the rank at every chunk start
        unsigned* out = tab.bm_arena + tab.bm_off[row];
        const int nch = chunks_of(nw);
        for (int c = warp; c < nch; c += DC_WARPS) {
            const int w = (c << 5) + lane;
            const unsigned word = (w < nw) ? bm[w] : 0u;
            if (w < nw) out[w] = word;
            int pc = __popc(word);
            for (int d = 16; d > 0; d >>= 1) pc += __shfl_xor_sync(0xffffffffu, pc, d);
            if (lane == 0) chunk[c] = pc;
        }
        __syncthreads();
        const int cpt = (nch + DC_THREADS - 1) / DC_THREADS;
        const int c_lo = min(nch, tid * cpt), c_hi = min(nch, c_lo + cpt);
        int local = 0;
        for (int c = c_lo; c < c_hi; ++c) local += chunk[c];
        int total;
        int run = block_excl_scan<DC_THREADS>(local, ws, total);
        for (int c = c_lo; c < c_hi; ++c) { out[nw + c] = (unsigned)run; run += chunk[c]; }
        if (tid == 0) tab.cnt[row] = total;
    }
}

// ---------------------------------------------------------------------------------------
// numeric, warp per row
// ---------------------------------------------------------------------------------------
// CEIL = true: the same walk over rows, entries and B rows with the workspace stripped (Sec. 7.2,
// iteration-only lower bound); the gathered indices and products go into two checksums.
template <typename T, bool CEIL>
__global__ void __launch_bounds__(DW_THREADS) dense_num_warp_kernel(DevCtl* __restrict__ ctl, int bmw, int accw, Csr A, Csr B, RowTables tab,
                                                                    const i64* __restrict__ rowptr, int* __restrict__ Ccrd,
                                                                    T* __restrict__ Cval, u64* __restrict__ chk_idx,
                                                                    double* __restrict__ chk_val) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    if (ctl->status != 0) return;
    const int n = ctl->n_warp_rows;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // per warp: a table of bmw bitmap words, each with the number of outputs before it (one load
    // ranks a column), and accw values (sized from the widest / largest row of this launch)
    uint2* tbl = reinterpret_cast<uint2*>(smem_raw) + warp * bmw;
    T* acc = reinterpret_cast<T*>(reinterpret_cast<uint2*>(smem_raw) + DW_WARPS * bmw) + warp * accw;
    const T* __restrict__ Aval = (const T*)A.val;
    const T* __restrict__ Bval = (const T*)B.val;
    if (!CEIL)
        for (int w = lane; w < bmw; w += 32) tbl[w] = make_uint2(0u, 0u);   // every row leaves its table clear
    __syncwarp();
    u64 my_idx = 0;
    double my_val = 0.0;
    for (;;) {
        int r = 0;
        if (lane == 0) r = atomicAdd(&ctl->work_counter[(CEIL ? CEIL_SLOT : NUM_SLOT) + CLS_DENSE_WARP], 1);
        r = __shfl_sync(0xffffffffu, r, 0);
        if (r >= n) break;
        const int row = tab.warp_rows[r];
        const int base = tab.jmin[row];
        const int nw = min((tab.jmax[row] - base) / 32 + 1, bmw);
        const unsigned span = (unsigned)nw * 32u;
        const i64 ps = A.pos[row], pe = A.pos[row + 1];
        const i64 out0 = rowptr[row];
        const int cnt = min((int)(rowptr[row + 1] - out0), accw);
        const i64 slot = tab.bm_off[row];
        const bool compact = (slot & BM_COMPACT) != 0;
        const int nzw = (int)((slot & ~BM_COMPACT) >> BM_NZW_SHIFT);
        const unsigned* src = tab.bm_arena + (slot & BM_OFF_MASK);
        const uint2* src2 = reinterpret_cast<const uint2*>(src);
        if (CEIL) {
            // no workspace to set up
        } else if (compact) {
            // the saved non-empty words in column order: ranks by a running prefix of their bit counts
            int carry = 0;
            for (int i0 = 0; i0 < nzw; i0 += 32) {
                const int i = i0 + lane;
                const uint2 e = (i < nzw) ? src2[i] : make_uint2(0u, 0u);
                const int c = __popc(e.x);
                const int incl = warp_incl_scan(c);
                if (i < nzw && e.y < (unsigned)nw) tbl[e.y] = make_uint2(e.x, (unsigned)(carry + incl - c));
                carry += __shfl_sync(0xffffffffu, incl, 31);
            }
        } else {
            // the whole bitmap; rank of each word's first bit = chunk rank + prefix inside the chunk
            for (int w0 = 0; w0 < nw; w0 += 32) {
                const int w = w0 + lane;
                const unsigned word = (w < nw) ? src[w] : 0u;
                const int c = __popc(word);
                const int incl = warp_incl_scan(c);
                if (w < nw) tbl[w] = make_uint2(word, src[nw + (w0 >> 5)] + (unsigned)(incl - c));
            }
        }
        if (!CEIL)
            for (int x = lane; x < cnt; x += 32) acc[x] = 0;
        __syncwarp();
        // one product into the workspace: rank of its column, then add (plain when no other lane can
        // hold the same column, atomic otherwise); stripped to the checksums when CEIL
        auto put = [&](unsigned rel, T prod, bool shared_slot) {
            if (CEIL) {
                if (rel != 0xffffffffu) { my_idx += (u64)(rel + (unsigned)base); my_val += (double)prod; }
            } else if (rel < span) {
                const uint2 t = tbl[rel >> 5];
                const int slot_ = (int)t.y + __popc(t.x & ((1u << (rel & 31)) - 1u));
                if (slot_ < accw) {
                    if (shared_slot) atomicAdd(&acc[slot_], prod);
                    else acc[slot_] = add_rn(acc[slot_], prod);
                }
            }
        };
        const int gs = pick_group_size(tab.ub[row], pe - ps, 1);
        if (gs == 32) {
            // one A entry at a time, lanes across its B row: distinct columns, no atomics,
            // every output summed in loop order
            // (the entries' descriptors are fetched 32 at a time, one per lane, and the first 32
            // elements of two B rows are loaded before either is consumed, to keep loads in flight)
            for (i64 p0 = ps; p0 < pe; p0 += 32) {
                i64 my_qs = 0;
                int my_len = 0;
                T my_a = 0;
                if (p0 + lane < pe) {
                    const int k = __ldg(A.crd + p0 + lane);
                    if ((unsigned)k < (unsigned)B.nrows) {
                        my_qs = __ldg(B.pos + k);
                        my_len = (int)(__ldg(B.pos + k + 1) - my_qs);
                    }
                    my_a = __ldg(Aval + p0 + lane);
                }
                const int nE = (int)min((i64)32, pe - p0);
                for (int e = 0; e < nE; e += 2) {
                    const i64 qs0 = __shfl_sync(0xffffffffu, my_qs, e), qs1 = __shfl_sync(0xffffffffu, my_qs, (e + 1) & 31);
                    const int len0 = __shfl_sync(0xffffffffu, my_len, e);
                    const int len1 = (e + 1 < nE) ? __shfl_sync(0xffffffffu, my_len, (e + 1) & 31) : 0;
                    const T a0 = __shfl_sync(0xffffffffu, my_a, e), a1 = __shfl_sync(0xffffffffu, my_a, (e + 1) & 31);
                    unsigned rel0 = 0xffffffffu, rel1 = 0xffffffffu;
                    T v0 = 0, v1 = 0;
                    if (lane < len0) { rel0 = (unsigned)(__ldg(B.crd + qs0 + lane) - base); v0 = __ldg(Bval + qs0 + lane); }
                    if (lane < len1) { rel1 = (unsigned)(__ldg(B.crd + qs1 + lane) - base); v1 = __ldg(Bval + qs1 + lane); }
                    // entry e
                    put(rel0, mul_rn(a0, v0), false);
                    for (int t = lane + 32; t < len0; t += 32)
                        put((unsigned)(__ldg(B.crd + qs0 + t) - base), mul_rn(a0, __ldg(Bval + qs0 + t)), false);
                    __syncwarp();
                    // entry e + 1
                    put(rel1, mul_rn(a1, v1), false);
                    for (int t = lane + 32; t < len1; t += 32)
                        put((unsigned)(__ldg(B.crd + qs1 + t) - base), mul_rn(a1, __ldg(Bval + qs1 + t)), false);
                    __syncwarp();
                }
            }
        } else {
            // short B rows: several A entries in flight, so slots can collide -> atomics
            const int g = lane / gs, gl = lane % gs, ng = 32 / gs;
            for (i64 p = ps + g; p < pe; p += ng) {
                const int k = __ldg(A.crd + p);
                if ((unsigned)k >= (unsigned)B.nrows) continue;
                const i64 qs = __ldg(B.pos + k);
                const int len = (int)(__ldg(B.pos + k + 1) - qs);
                const T a = __ldg(Aval + p);
                for (int t = gl; t < len; t += gs)
                    put((unsigned)(__ldg(B.crd + qs + t) - base), mul_rn(a, __ldg(Bval + qs + t)), true);
            }
            __syncwarp();
        }
        if (CEIL) continue;
        // copy out: values are already in output order; set bits give the coordinates; the table
        // words the row used are cleared on the way
        for (int x = lane; x < cnt; x += 32) Cval[out0 + x] = acc[x];
        if (compact) {
            for (int i = lane; i < nzw; i += 32) {
                const uint2 e = src2[i];
                if (e.y >= (unsigned)nw) continue;
                unsigned word = e.x;
                i64 o = out0 + tbl[e.y].y;
                tbl[e.y] = make_uint2(0u, 0u);
                while (word) {
                    const int b = __ffs(word) - 1;
                    word &= word - 1;
                    Ccrd[o++] = base + (int)(e.y << 5) + b;
                }
            }
        } else {
            for (int w = lane; w < nw; w += 32) {
                const uint2 t = tbl[w];
                unsigned word = t.x;
                i64 o = out0 + t.y;
                tbl[w] = make_uint2(0u, 0u);
                while (word) {
                    const int b = __ffs(word) - 1;
                    word &= word - 1;
                    Ccrd[o++] = base + (w << 5) + b;
                }
            }
        }
        __syncwarp();
    }
    if (CEIL) {
        for (int d = 16; d > 0; d >>= 1) {
            my_idx += __shfl_xor_sync(0xffffffffu, my_idx, d);
            my_val += __shfl_xor_sync(0xffffffffu, my_val, d);
        }
        if (lane == 0) { atomicAdd(chk_idx, my_idx); atomicAdd(chk_val, my_val); }
    }
}

// ---------------------------------------------------------------------------------------
// numeric, CTA units.  A unit is a row, or an equal share of the A entries of a row with very
// many products.  Every unit streams its B rows once, whole.  Outputs with rank < CAP accumulate
// in shared memory; outputs beyond accumulate straight into the row's value segment in global
// memory (zeroed beforehand), which keeps any row to a single pass whatever its output count.
// ---------------------------------------------------------------------------------------
constexpr int DN_ENTRIES = 768;      // A entries whose descriptors are staged per round
constexpr int DN_TILE = 256;         // products a warp takes per fetch

// CEIL = true is the same traversal with the workspace stripped (the iteration-only lower bound of
// Sec. 7.2): units, descriptor rounds, product tiles and gathers as below, but no bitmap, no rank
// and no accumulation; every gathered column index and product is folded into two checksums.
template <typename T, bool CEIL>
__global__ void __launch_bounds__(DN_THREADS, 2) dense_num_cta_kernel(DevCtl* __restrict__ ctl, int smem_words, int CAP, i64 unit_products,
                                                                   Csr A, Csr B, RowTables tab, const i64* __restrict__ rowptr,
                                                                   int* __restrict__ Ccrd, T* __restrict__ Cval,
                                                                   u64* __restrict__ chk_idx, double* __restrict__ chk_val) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* acc = reinterpret_cast<T*>(smem_raw);                                        // CAP
    // per bitmap word: .x = the word, .y = outputs of the row before it (one load gives a rank)
    uint2* bmr = reinterpret_cast<uint2*>(acc + CAP);                                // smem_words
    // staged descriptors of up to DN_ENTRIES A entries: B-row start, A value, running product count
    i64* d_qs = reinterpret_cast<i64*>(smem_raw + ((sizeof(T) * (size_t)CAP + 8 * (size_t)smem_words + 15) & ~(size_t)15));
    T* d_a = reinterpret_cast<T*>(d_qs + DN_ENTRIES);
    int* d_pre = reinterpret_cast<int*>(d_a + DN_ENTRIES);                           // DN_ENTRIES + 1
    __shared__ int s_next, s_tile;
    __shared__ int ws[33];
    if (ctl->status != 0) return;
    const int n_units = ctl->n_units;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T* __restrict__ Aval = (const T*)A.val;
    const T* __restrict__ Bval = (const T*)B.val;
    if (!CEIL)
        for (int x = tid; x < CAP; x += DN_THREADS) acc[x] = 0;
    u64 my_idx = 0;
    double my_val = 0.0;

    for (;;) {
        __syncthreads();
        if (tid == 0) s_next = atomicAdd(&ctl->work_counter[(CEIL ? CEIL_SLOT : NUM_SLOT) + CLS_DENSE_CTA], 1);
        __syncthreads();
        const int u = s_next;
        if (u >= n_units) break;
        const int row = tab.unit_row[u];
        const int uidx = u - tab.row_unit0[row];
        const int nun = dense_units_of_row(tab.ub[row], unit_products);
        const int base = tab.jmin[row], last = tab.jmax[row];
        const int nw = min((last - base) / 32 + 1, smem_words);
        const int nch = chunks_of(nw);
        const unsigned span_bits = (unsigned)nw * 32u;
        const i64 out0 = rowptr[row];
        const int cnt = (int)(rowptr[row + 1] - out0);
        const i64 ps = A.pos[row], pe = A.pos[row + 1];
        const i64 e_lo = ps + (pe - ps) * uidx / nun, e_hi = ps + (pe - ps) * (uidx + 1) / nun;
        T* const gacc = Cval + out0;
        if (!CEIL && nun == 1)                          // outputs beyond the shared-memory part start at zero
            for (int x = CAP + tid; x < cnt; x += DN_THREADS) gacc[x] = 0;

        // the row's bitmap with the rank of every word's first bit (the symbolic pass saved the
        // rank at every chunk start).  A warp takes eight chunks at a time, all loads first.
        const unsigned* src = tab.bm_arena + tab.bm_off[row];
        for (int c0 = warp; !CEIL && c0 < nch; c0 += DN_WARPS * 8) {
            unsigned word[8], rank_c[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) {
                const int c = c0 + x * DN_WARPS, w = (c << 5) + lane;
                word[x] = (w < nw) ? src[w] : 0u;
                rank_c[x] = (c < nch) ? src[nw + c] : 0u;
            }
#pragma unroll
            for (int x = 0; x < 8; ++x) {
                const int c = c0 + x * DN_WARPS, w = (c << 5) + lane;
                const int pc = __popc(word[x]);
                const int incl = warp_incl_scan(pc);
                if (w < nw) bmr[w] = make_uint2(word[x], rank_c[x] + (unsigned)(incl - pc));
            }
        }
        __syncthreads();

#define SPWS_DENSE_ADD(REL, VAL)                                                                          \
        if (CEIL) {                                                                                       \
            if ((REL) != 0xffffffffu) { my_idx += (u64)((REL) + (unsigned)base); my_val += (double)(VAL); } \
        } else if ((REL) < span_bits) {                                                                   \
            const uint2 br_ = bmr[(REL) >> 5];                                                            \
            const int r_ = (int)br_.y + __popc(br_.x & ((1u << ((REL) & 31)) - 1u));                      \
            if (r_ < CAP) atomicAdd(&acc[r_], (VAL));                                                     \
            else if (r_ < cnt) atomicAdd(gacc + r_, (VAL));                                               \
        }

        const float avg_len = (float)tab.ub[row] / fmaxf(1.0f, (float)(pe - ps));
        const bool long_rows = avg_len >= 64.0f;
        {
            // Rounds of up to DN_ENTRIES A entries.  Step 1: every thread fetches the descriptors
            // of two entries; a block scan turns the B-row lengths into a running product count.
            // Step 2: warps pull tiles of DN_TILE consecutive products of that stream, so the
            // work is shared evenly however long the individual B rows are.
            for (i64 e0 = e_lo; e0 < e_hi; e0 += DN_ENTRIES) {
                const int nE = (int)min((i64)DN_ENTRIES, e_hi - e0);
                int len2[2] = {0, 0};
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    const int i = 2 * tid + x;
                    if (i < nE) {
                        const int k = __ldg(A.crd + e0 + i);
                        i64 qs = 0;
                        if ((unsigned)k < (unsigned)B.nrows) {
                            qs = __ldg(B.pos + k);
                            len2[x] = (int)(__ldg(B.pos + k + 1) - qs);
                        }
                        d_qs[i] = qs;
                        d_a[i] = __ldg(Aval + e0 + i);
                    }
                }
                int total;
                const int excl = block_excl_scan<DN_THREADS>(len2[0] + len2[1], ws, total);
                if (2 * tid < nE) d_pre[2 * tid] = excl;
                if (2 * tid + 1 < nE) d_pre[2 * tid + 1] = excl + len2[0];
                if (tid == 0) { d_pre[nE] = total; s_tile = 0; }
                __syncthreads();
                // Every warp walks the product stream tile by tile.  The loads of a step are
                // issued before the previous step is ranked and added, so gather latency and
                // accumulation overlap inside a warp as well as across warps.
                int t0 = 0, t1 = 0, e = 0;              // stream position, end of the tile in hand, entry at t0
                auto next_tile = [&]() -> bool {
                    int s = 0;
                    if (lane == 0) s = atomicAdd(&s_tile, DN_TILE);
                    t0 = __shfl_sync(0xffffffffu, s, 0);
                    if (t0 >= total) return false;
                    t1 = min(total, t0 + DN_TILE);
                    int lo = 0, hi = nE;                // the last entry whose running count is <= t0
                    while (hi - lo > 1) {
                        const int mid = (lo + hi) >> 1;
                        if (d_pre[mid] <= t0) lo = mid; else hi = mid;
                    }
                    e = lo;
                    return true;
                };
                if (long_rows) {
                    // a step = up to 128 consecutive products of one B row, four per lane
                    auto fetch = [&](unsigned (&rel)[4], T (&b)[4], T& a) -> bool {
                        if (t0 >= t1 && !next_tile()) return false;
                        while (d_pre[e + 1] <= t0) ++e;
                        const int off = t0 - d_pre[e];
                        const int n = min(min(t1, d_pre[e + 1]) - t0, 128);
                        const int* __restrict__ ck = B.crd + d_qs[e] + off;
                        const T* __restrict__ vk = Bval + d_qs[e] + off;
                        a = d_a[e];
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            const int idx = lane + 32 * x;
                            rel[x] = idx < n ? (unsigned)(__ldg(ck + idx) - base) : 0xffffffffu;
                            b[x] = idx < n ? __ldg(vk + idx) : (T)0;
                        }
                        t0 += n;
                        return true;
                    };
                    unsigned relc[4] = {0, 0, 0, 0}, reln[4] = {0, 0, 0, 0};
                    T bc[4] = {0, 0, 0, 0}, bn[4] = {0, 0, 0, 0};
                    T ac = 0, an = 0;
                    bool have = fetch(relc, bc, ac);
                    while (have) {
                        const bool more = fetch(reln, bn, an);
#pragma unroll
                        for (int x = 0; x < 4; ++x) { SPWS_DENSE_ADD(relc[x], ac * bc[x]) }
#pragma unroll
                        for (int x = 0; x < 4; ++x) { relc[x] = reln[x]; bc[x] = bn[x]; }
                        ac = an;
                        have = more;
                    }
                } else {
                    // short B rows: a step = 64 consecutive products of the stream, two per lane;
                    // every lane advances its own entry index across row boundaries
                    int my_e = 0;
                    auto fetch = [&](unsigned (&rel)[2], T (&b)[2], T (&a)[2]) -> bool {
                        if (t0 >= t1) {
                            if (!next_tile()) return false;
                            my_e = e;
                        }
#pragma unroll
                        for (int x = 0; x < 2; ++x) {
                            const int t = t0 + lane + 32 * x;
                            rel[x] = 0xffffffffu;
                            b[x] = 0;
                            a[x] = 0;
                            if (t < t1) {
                                while (d_pre[my_e + 1] <= t) ++my_e;
                                const i64 q = d_qs[my_e] + (t - d_pre[my_e]);
                                a[x] = d_a[my_e];
                                rel[x] = (unsigned)(__ldg(B.crd + q) - base);
                                b[x] = __ldg(Bval + q);
                            }
                        }
                        t0 = min(t1, t0 + 64);
                        return true;
                    };
                    unsigned relc[2] = {0, 0}, reln[2] = {0, 0};
                    T bc[2] = {0, 0}, bn[2] = {0, 0}, ac[2] = {0, 0}, an[2] = {0, 0};
                    bool have = fetch(relc, bc, ac);
                    while (have) {
                        const bool more = fetch(reln, bn, an);
#pragma unroll
                        for (int x = 0; x < 2; ++x) { SPWS_DENSE_ADD(relc[x], ac[x] * bc[x]) }
#pragma unroll
                        for (int x = 0; x < 2; ++x) { relc[x] = reln[x]; bc[x] = bn[x]; ac[x] = an[x]; }
                        have = more;
                    }
                }
                __syncthreads();
            }
        }
#undef SPWS_DENSE_ADD

        // copy out the shared-memory part of the values (the coordinates are written by
        // dense_emit_crd_kernel)
        const int n_smem = CEIL ? 0 : min(cnt, CAP);
        if (nun == 1) {
            for (int x = tid; x < n_smem; x += DN_THREADS) { gacc[x] = acc[x]; acc[x] = 0; }
        } else {
            for (int x = tid; x < n_smem; x += DN_THREADS) {
                const T v = acc[x];
                acc[x] = 0;
                if (v != (T)0) atomicAdd(gacc + x, v);
            }
        }
    }
    if (CEIL) {
        for (int d = 16; d > 0; d >>= 1) {
            my_idx += __shfl_xor_sync(0xffffffffu, my_idx, d);
            my_val += __shfl_xor_sync(0xffffffffu, my_val, d);
        }
        if (lane == 0) { atomicAdd(chk_idx, my_idx); atomicAdd(chk_val, my_val); }
    }
}

// Coordinates of the CTA-unit rows, and the clearing of the value segments that several units
// add into.  Runs before the accumulation kernel.  The saved bitmap carries the rank at every
// 32-word chunk, so any stretch of a row can be expanded on its own: unit c of a row's n units
// takes the c-th n-th of the row's 128-word groups, which spreads a hub row over as many warps as
// it has units.  A warp takes one group at a time, four consecutive words per lane (one 16-byte
// load); the lanes' bit counts are scanned once per group.  Unless the non-empty words of a group
// are half full on average, every lane expands its own words into a small shared-memory stage at
// their ranks and the stage goes out with contiguous stores; otherwise the warp takes one word
// per step with a lane per bit.
constexpr int DE_THREADS = 256;
constexpr int DE_WARPS = DE_THREADS / 32;
constexpr int DE_STAGE = 2048;       // coordinates a warp stages at once (128 words, 16 bits each on average)

template <typename T>
__global__ void __launch_bounds__(DE_THREADS) dense_emit_crd_kernel(DevCtl* __restrict__ ctl, i64 unit_products, RowTables tab,
                                                                    const i64* __restrict__ rowptr, int* __restrict__ Ccrd,
                                                                    T* __restrict__ Cval) {
    __shared__ unsigned short s_stage[DE_WARPS][DE_STAGE];
    if (ctl->status != 0) return;
    const int n_units = ctl->n_units;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned short* stage = s_stage[warp];
    for (;;) {
        int u = 0;
        if (lane == 0) u = atomicAdd(&ctl->work_counter[EMIT_SLOT], 1);
        u = __shfl_sync(0xffffffffu, u, 0);
        if (u >= n_units) break;
        const int row = tab.unit_row[u];
        const int uidx = u - tab.row_unit0[row];
        const int nun = dense_units_of_row(tab.ub[row], unit_products);
        const int base = tab.jmin[row];
        const int nw = (tab.jmax[row] - base) / 32 + 1;
        const int nch = chunks_of(nw);
        const int ng = (nch + 3) >> 2;                                  // groups of four chunks = 128 words
        const int g_lo = (int)((i64)ng * uidx / nun), g_hi = (int)((i64)ng * (uidx + 1) / nun);
        const unsigned* src = tab.bm_arena + tab.bm_off[row];
        const uint4* src4 = reinterpret_cast<const uint4*>(src);         // slots are 16-byte aligned
        const i64 out0 = rowptr[row];
        const int cnt_row = (int)(rowptr[row + 1] - out0);
        const bool clear = nun > 1;                                      // several units add into this row's values

        // words 128 g + 4 lane .. + 3 (zero past the end of the bitmap) and the ranks at both ends of group g
        auto load_group = [&](int g, uint4& w, int& r0, int& r1) {
            w = make_uint4(0u, 0u, 0u, 0u);
            r0 = r1 = cnt_row;
            if (g >= g_hi) return;
            const int w0 = (g << 7) + (lane << 2);
            if (w0 < nw) {
                w = src4[(g << 5) + lane];
                if (w0 + 1 >= nw) w.y = 0u;
                if (w0 + 2 >= nw) w.z = 0u;
                if (w0 + 3 >= nw) w.w = 0u;
            }
            r0 = (int)src[nw + (g << 2)];
            if ((g << 2) + 4 < nch) r1 = (int)src[nw + (g << 2) + 4];
        };
        uint4 w, wn;
        int r0, r1, r0n, r1n;
        load_group(g_lo, w, r0, r1);
        for (int g = g_lo; g < g_hi; ++g) {
            load_group(g + 1, wn, r0n, r1n);                             // next group's loads fly during this expansion
            const int n = r1 - r0;
            if (n > 0) {
                const int p = __popc(w.x) + __popc(w.y) + __popc(w.z) + __popc(w.w);
                const int e = warp_incl_scan(p) - p;
                const i64 o = out0 + r0;
                const unsigned m0 = __ballot_sync(0xffffffffu, w.x != 0u), m1 = __ballot_sync(0xffffffffu, w.y != 0u);
                const unsigned m2 = __ballot_sync(0xffffffffu, w.z != 0u), m3 = __ballot_sync(0xffffffffu, w.w != 0u);
                const int nzw = __popc(m0) + __popc(m1) + __popc(m2) + __popc(m3);
                if (n <= DE_STAGE && n < 16 * nzw) {
                    // every lane expands its own four words into the stage at their ranks (as 16-bit
                    // offsets from the group's first column), then the stage goes out with
                    // contiguous stores
                    int slot = e;
                    auto expand = [&](unsigned word, int off0) {
                        while (word) {
                            const int b = __ffs(word) - 1;
                            word &= word - 1;
                            stage[slot++] = (unsigned short)(off0 + b);
                        }
                    };
                    const int off = lane << 7;
                    expand(w.x, off); expand(w.y, off + 32); expand(w.z, off + 64); expand(w.w, off + 96);
                    __syncwarp();
                    const int gcol0 = base + (g << 12);
                    for (int y = lane; y < n; y += 32) Ccrd[o + y] = gcol0 + (int)stage[y];
                    __syncwarp();
                } else {
                    // half-full words or fuller: the warp expands one non-empty word per step, lane
                    // b testing bit b, so the word's outputs leave as one contiguous store
                    const unsigned below = (1u << lane) - 1u;
                    const int gcol = base + (g << 12) + lane;
                    auto spread = [&](unsigned mine, int rank_mine, unsigned m, int x) {
                        while (m) {
                            const int L = __ffs(m) - 1;
                            m &= m - 1;
                            const unsigned word = __shfl_sync(0xffffffffu, mine, L);
                            const int at = __shfl_sync(0xffffffffu, rank_mine, L);
                            if ((word >> lane) & 1u) Ccrd[o + at + __popc(word & below)] = gcol + (((L << 2) + x) << 5);
                        }
                    };
                    const int e1 = e + __popc(w.x), e2 = e1 + __popc(w.y), e3 = e2 + __popc(w.z);
                    spread(w.x, e, m0, 0); spread(w.y, e1, m1, 1); spread(w.z, e2, m2, 2); spread(w.w, e3, m3, 3);
                }
                if (clear)
                    for (int y = lane; y < n; y += 32) Cval[o + y] = (T)0;
            }
            w = wn; r0 = r0n; r1 = r1n;
        }
    }
}

// ---------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------
static int persistent_grid(const LaunchCtx& c, int per_sm, i64 work) {
    i64 grid = (i64)c.sm_count * (per_sm > 0 ? per_sm : 1);
    if (work >= 0 && work < grid) grid = work > 0 ? work : 1;
    return (int)grid;
}

cudaError_t launch_dense_sym_warp(const LaunchCtx& c, const Csr& A, const Csr& B) {
    int per_sm = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, dense_sym_warp_kernel, DW_THREADS, 0);
    if (e != cudaSuccess) return e;
    dense_sym_warp_kernel<<<persistent_grid(c, per_sm, -1), DW_THREADS, 0, c.stream>>>(c.ctl, A, B, c.tab);
    ++c.launches;
    return cudaGetLastError();
}

cudaError_t launch_dense_sym_cta(const LaunchCtx& c, const Csr& A, const Csr& B) {
    const size_t smem = (size_t)c.dense_smem_words * 4 + (size_t)(c.dense_smem_words / 32 + 1) * 4;
    cudaError_t e;
    int per_sm = 0;
    if ((e = cudaFuncSetAttribute(dense_sym_cta_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, dense_sym_cta_kernel, DC_THREADS, smem)) != cudaSuccess) return e;
    dense_sym_cta_kernel<<<persistent_grid(c, per_sm, -1), DC_THREADS, smem, c.stream>>>(c.ctl, c.dense_smem_words, A, B, c.tab, c.bw);
    ++c.launches;
    return cudaGetLastError();
}

template <typename T, bool CEIL>
static cudaError_t num_warp_t(const LaunchCtx& c, int n_host, int bmw, int accw, const Csr& A, const Csr& B, const i64* rowptr, int* Ccrd,
                              void* Cval, u64* chk_idx, double* chk_val) {
    int per_sm = 0;
    const size_t smem = (size_t)DW_WARPS * (sizeof(T) * (size_t)accw + 8 * (size_t)bmw);
    cudaError_t e;
    auto k = dense_num_warp_kernel<T, CEIL>;
    if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, DW_THREADS, smem)) != cudaSuccess) return e;
    const i64 work = n_host >= 0 ? ((i64)n_host + DW_WARPS - 1) / DW_WARPS : -1;
    k<<<persistent_grid(c, per_sm, work), DW_THREADS, smem, c.stream>>>(c.ctl, bmw, accw, A, B, c.tab, rowptr, Ccrd, (T*)Cval, chk_idx, chk_val);
    ++c.launches;
    return cudaGetLastError();
}

cudaError_t launch_dense_num_warp(const LaunchCtx& c, int n_host, int max_span_words, int max_cnt, const Csr& A, const Csr& B,
                                  const i64* rowptr, int* Ccrd, void* Cval, u64* chk_idx, double* chk_val) {
    // bitmap words reserved per warp: the widest dense row of this pass, at most the class limit
    int bmw = max_span_words > 0 ? ((max_span_words + 31) & ~31) : DENSE_WARP_BM_WORDS;
    if (bmw > DENSE_WARP_BM_WORDS) bmw = DENSE_WARP_BM_WORDS;
    int accw = max_cnt > 0 ? ((max_cnt + 31) & ~31) : DENSE_WARP_ACC;     // values reserved per warp
    if (accw > DENSE_WARP_ACC) accw = DENSE_WARP_ACC;
    if (chk_idx)      // same launch shape (shared memory reserved, hence occupancy) as the full kernel
        return c.is_f64 ? num_warp_t<double, true>(c, n_host, bmw, accw, A, B, rowptr, Ccrd, Cval, chk_idx, chk_val)
                        : num_warp_t<float, true>(c, n_host, bmw, accw, A, B, rowptr, Ccrd, Cval, chk_idx, chk_val);
    return c.is_f64 ? num_warp_t<double, false>(c, n_host, bmw, accw, A, B, rowptr, Ccrd, Cval, nullptr, nullptr)
                    : num_warp_t<float, false>(c, n_host, bmw, accw, A, B, rowptr, Ccrd, Cval, nullptr, nullptr);
}

template <typename T, bool CEIL>
static cudaError_t num_cta_t(const LaunchCtx& c, int phase, int n_units_host, int words, i64 total_products, const Csr& A,
                             const Csr& B, const i64* rowptr, int* Ccrd, void* Cval, u64* chk_idx, double* chk_val) {
    const int CAP = c.prm.unit_outputs;
    const i64 unit_products = dense_unit_products(total_products);
    const size_t smem = ((sizeof(T) * (size_t)CAP + (size_t)words * 8 + 15) & ~(size_t)15) +
                        (size_t)DN_ENTRIES * (8 + sizeof(T)) + (size_t)(DN_ENTRIES + 1) * 4 + 16;
    cudaError_t e;
    int per_sm = 0;
    auto k = dense_num_cta_kernel<T, CEIL>;
    if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, DN_THREADS, smem)) != cudaSuccess) return e;
    if (phase == 0) {
        // units are dealt out dynamically, so the grid is what is resident at once
        int emit_per_sm = 0;
        if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&emit_per_sm, dense_emit_crd_kernel<T>, DE_THREADS, 0)) != cudaSuccess) return e;
        const i64 work = n_units_host >= 0 ? ((i64)n_units_host + DE_WARPS - 1) / DE_WARPS : -1;
        dense_emit_crd_kernel<T><<<persistent_grid(c, emit_per_sm, work), DE_THREADS, 0, c.stream>>>(c.ctl, unit_products, c.tab, rowptr, Ccrd, (T*)Cval);
    } else {
        k<<<persistent_grid(c, per_sm, n_units_host), DN_THREADS, smem, c.stream>>>(c.ctl, words, CAP, unit_products, A, B, c.tab,
                                                                                 rowptr, Ccrd, (T*)Cval, chk_idx, chk_val);
    }
    ++c.launches;
    return cudaGetLastError();
}

cudaError_t launch_dense_num_cta(const LaunchCtx& c, int phase, int n_units_host, int max_span_words, i64 total_products,
                                 const Csr& A, const Csr& B, const i64* rowptr, int* Ccrd, void* Cval, u64* chk_idx, double* chk_val) {
    int words = max_span_words > 0 ? max_span_words : c.dense_smem_words;
    words = (words + 31) & ~31;
    if (chk_idx)      // same launch shape as the full kernel
        return c.is_f64 ? num_cta_t<double, true>(c, 1, n_units_host, words, total_products, A, B, rowptr, Ccrd, Cval, chk_idx, chk_val)
                        : num_cta_t<float, true>(c, 1, n_units_host, words, total_products, A, B, rowptr, Ccrd, Cval, chk_idx, chk_val);
    return c.is_f64 ? num_cta_t<double, false>(c, phase, n_units_host, words, total_products, A, B, rowptr, Ccrd, Cval, nullptr, nullptr)
                    : num_cta_t<float, false>(c, phase, n_units_host, words, total_products, A, B, rowptr, Ccrd, Cval, nullptr, nullptr);
}

}  // namespace spws
