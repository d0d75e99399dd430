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
//   CTA units    : any span up to 2^20 columns.  A row is cut into units of `unit_outputs`
//              consecutive outputs (rank ranges), so units carry equal output counts however
//              skewed the columns are; hub rows spread over many CTAs and write disjoint,
//              ordered pieces of the row.  Shared-memory atomics combine the CTA's warps.
#include "common.cuh"

namespace spws {

constexpr int DW_THREADS = 256;            // warp-per-row kernels: 8 warps per CTA
constexpr int DW_WARPS = DW_THREADS / 32;
constexpr int DC_THREADS = 256;            // symbolic CTA kernel
constexpr int DC_WARPS = DC_THREADS / 32;
constexpr int DN_THREADS = 1024;           // numeric CTA kernel
constexpr int DN_WARPS = DN_THREADS / 32;

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
    if (ctl->status != 0) return;
    int off, n;
    class_range(ctl, CLS_DENSE_WARP, off, n);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned* bm = s_bm[warp];
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
        for (int w = lane; w < nw; w += 32) bm[w] = 0;
        __syncwarp();
        const int gs = pick_group_size(tab.ub[row], pe - ps, 1);
        const int g = lane / gs, gl = lane % gs, ng = 32 / gs;
        for (i64 p = ps + g; p < pe; p += ng) {
            const int k = __ldg(A.crd + p);
            if ((unsigned)k >= (unsigned)B.nrows) continue;
            const i64 qs = __ldg(B.pos + k);
            const int len = (int)(__ldg(B.pos + k + 1) - qs);
            const int* __restrict__ ck = B.crd + qs;
            for (int t = gl; t < len; t += gs) {
                const unsigned rel = (unsigned)(__ldg(ck + t) - base);
                if (rel < span) atomicOr(&bm[rel >> 5], 1u << (rel & 31));
            }
        }
        __syncwarp();
        unsigned* out = tab.bm_arena + tab.bm_off[row];
        int carry = 0;
        for (int w0 = 0; w0 < nw; w0 += 32) {
            const int w = w0 + lane;
            const unsigned word = (w < nw) ? bm[w] : 0u;
            if (w < nw) out[w] = word;
            int c = __popc(word);
            for (int d = 16; d > 0; d >>= 1) c += __shfl_xor_sync(0xffffffffu, c, d);
            if (lane == 0) out[nw + (w0 >> 5)] = (unsigned)carry;
            carry += c;
        }
        if (lane == 0) tab.cnt[row] = carry;
        __syncwarp();
    }
}

// ---------------------------------------------------------------------------------------
// symbolic, CTA per row (hub rows first: classes HUB and CTA are adjacent in perm)
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(DC_THREADS) dense_sym_cta_kernel(DevCtl* __restrict__ ctl, int smem_words, Csr A, Csr B, RowTables tab) {
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
template <typename T>
__global__ void __launch_bounds__(DW_THREADS) dense_num_warp_kernel(DevCtl* __restrict__ ctl, Csr A, Csr B, RowTables tab,
                                                                    const i64* __restrict__ rowptr, int* __restrict__ Ccrd,
                                                                    T* __restrict__ Cval) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    if (ctl->status != 0) return;
    const int n = ctl->n_warp_rows;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    T* acc = reinterpret_cast<T*>(smem_raw) + warp * DENSE_WARP_ACC;
    unsigned* bm = reinterpret_cast<unsigned*>(reinterpret_cast<T*>(smem_raw) + DW_WARPS * DENSE_WARP_ACC) + warp * DENSE_WARP_BM_WORDS;
    unsigned short* pre = reinterpret_cast<unsigned short*>(reinterpret_cast<unsigned*>(reinterpret_cast<T*>(smem_raw) + DW_WARPS * DENSE_WARP_ACC) +
                                                            DW_WARPS * DENSE_WARP_BM_WORDS) + warp * DENSE_WARP_BM_WORDS;
    const T* __restrict__ Aval = (const T*)A.val;
    const T* __restrict__ Bval = (const T*)B.val;
    for (;;) {
        int r = 0;
        if (lane == 0) r = atomicAdd(&ctl->work_counter[8 + CLS_DENSE_WARP], 1);
        r = __shfl_sync(0xffffffffu, r, 0);
        if (r >= n) break;
        const int row = tab.warp_rows[r];
        const int base = tab.jmin[row];
        const int nw = (tab.jmax[row] - base) / 32 + 1;
        const unsigned span = (unsigned)nw * 32u;
        const i64 ps = A.pos[row], pe = A.pos[row + 1];
        const i64 out0 = rowptr[row];
        const int cnt = (int)(rowptr[row + 1] - out0);
        // reload the bitmap; rank of each word's first bit = chunk rank + prefix inside the chunk
        const unsigned* src = tab.bm_arena + tab.bm_off[row];
        for (int w0 = 0; w0 < nw; w0 += 32) {
            const int w = w0 + lane;
            const unsigned word = (w < nw) ? src[w] : 0u;
            const int c = __popc(word);
            const int incl = warp_incl_scan(c);
            if (w < nw) { bm[w] = word; pre[w] = (unsigned short)((int)src[nw + (w0 >> 5)] + incl - c); }
        }
        for (int x = lane; x < cnt; x += 32) acc[x] = 0;
        __syncwarp();
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
                    if (rel0 < span) {
                        const int slot = pre[rel0 >> 5] + __popc(bm[rel0 >> 5] & ((1u << (rel0 & 31)) - 1u));
                        if (slot < DENSE_WARP_ACC) acc[slot] = add_rn(acc[slot], mul_rn(a0, v0));
                    }
                    for (int t = lane + 32; t < len0; t += 32) {
                        const unsigned rel = (unsigned)(__ldg(B.crd + qs0 + t) - base);
                        if (rel < span) {
                            const int slot = pre[rel >> 5] + __popc(bm[rel >> 5] & ((1u << (rel & 31)) - 1u));
                            if (slot < DENSE_WARP_ACC) acc[slot] = add_rn(acc[slot], mul_rn(a0, __ldg(Bval + qs0 + t)));
                        }
                    }
                    __syncwarp();
                    // entry e + 1
                    if (rel1 < span) {
                        const int slot = pre[rel1 >> 5] + __popc(bm[rel1 >> 5] & ((1u << (rel1 & 31)) - 1u));
                        if (slot < DENSE_WARP_ACC) acc[slot] = add_rn(acc[slot], mul_rn(a1, v1));
                    }
                    for (int t = lane + 32; t < len1; t += 32) {
                        const unsigned rel = (unsigned)(__ldg(B.crd + qs1 + t) - base);
                        if (rel < span) {
                            const int slot = pre[rel >> 5] + __popc(bm[rel >> 5] & ((1u << (rel & 31)) - 1u));
                            if (slot < DENSE_WARP_ACC) acc[slot] = add_rn(acc[slot], mul_rn(a1, __ldg(Bval + qs1 + t)));
                        }
                    }
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
                for (int t = gl; t < len; t += gs) {
                    const unsigned rel = (unsigned)(__ldg(B.crd + qs + t) - base);
                    if (rel < span) {
                        const int slot = pre[rel >> 5] + __popc(bm[rel >> 5] & ((1u << (rel & 31)) - 1u));
                        if (slot < DENSE_WARP_ACC) atomicAdd(&acc[slot], mul_rn(a, __ldg(Bval + qs + t)));
                    }
                }
            }
            __syncwarp();
        }
        // copy out: values are already in output order; set bits give the coordinates
        for (int x = lane; x < cnt; x += 32) Cval[out0 + x] = acc[x];
        for (int w = lane; w < nw; w += 32) {
            unsigned word = bm[w];
            i64 o = out0 + pre[w];
            while (word) {
                const int b = __ffs(word) - 1;
                word &= word - 1;
                Ccrd[o++] = base + (w << 5) + b;
            }
        }
        __syncwarp();
    }
}

// ---------------------------------------------------------------------------------------
// numeric, CTA units (row, rank range)
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ int nth_set_bit(unsigned word, int nth) {   // position of the nth (0-based) set bit
    for (int x = 0; x < nth; ++x) word &= word - 1;
    return __ffs(word) - 1;
}

// Plain lower bound by one lane (all lanes of a warp search different rows at once).
__device__ __forceinline__ int lane_lower_bound(const int* __restrict__ ck, int lo, int hi, int c) {
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(ck + mid) < c) lo = mid + 1; else hi = mid;
    }
    return lo;
}

constexpr int DN_ENTRIES = 1024;     // A entries examined per round
constexpr int DN_LONG = 2048;        // segments at least this long are walked by the whole CTA
constexpr int DN_LONG_CAP = 32;

template <typename T>
__global__ void __launch_bounds__(DN_THREADS) dense_num_cta_kernel(DevCtl* __restrict__ ctl, int smem_words, int CAP, Csr A, Csr B,
                                                                   RowTables tab, const i64* __restrict__ rowptr,
                                                                   int* __restrict__ Ccrd, T* __restrict__ Cval) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* acc = reinterpret_cast<T*>(smem_raw);                                        // CAP
    T* item_a = acc + CAP;                                                           // DN_ENTRIES
    i64* item_q = reinterpret_cast<i64*>(item_a + DN_ENTRIES);                       // DN_ENTRIES
    int* item_len = reinterpret_cast<int*>(item_q + DN_ENTRIES);                     // DN_ENTRIES
    unsigned* bm = reinterpret_cast<unsigned*>(item_len + DN_ENTRIES);               // smem_words
    short* pre = reinterpret_cast<short*>(bm + smem_words);                          // smem_words: rank of word start - r0
    __shared__ int s_next, s_ca, s_cb, s_w0, s_w1, s_c0, s_c1, s_items, s_fetch, s_nlong, s_sumlen;
    __shared__ int s_long[DN_LONG_CAP];
    if (ctl->status != 0) return;
    const int n_units = ctl->n_units;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T* __restrict__ Aval = (const T*)A.val;
    const T* __restrict__ Bval = (const T*)B.val;
    for (int x = tid; x < CAP; x += DN_THREADS) acc[x] = 0;

    for (;;) {
        __syncthreads();
        if (tid == 0) s_next = atomicAdd(&ctl->work_counter[8 + CLS_DENSE_CTA], 1);
        __syncthreads();
        const int u = s_next;
        if (u >= n_units) break;
        const int row = tab.unit_row[u];
        const int uidx = u - tab.row_unit0[row];
        const int base = tab.jmin[row], last = tab.jmax[row];
        const int nw = min((last - base) / 32 + 1, smem_words);
        const int nch = chunks_of(nw);
        const i64 out0 = rowptr[row];
        const int cnt = (int)(rowptr[row + 1] - out0);
        const int r0 = uidx * CAP;
        const int nout = min(CAP, cnt - r0);
        const int r1 = r0 + nout;
        const bool whole = (r0 == 0 && r1 == cnt);
        const i64 ps = A.pos[row], pe = A.pos[row + 1];
        const unsigned* src = tab.bm_arena + tab.bm_off[row];
        const int* cpre = reinterpret_cast<const int*>(src + nw);      // rank at every chunk start
        if (tid == 0) { s_ca = 0; s_cb = nch - 1; s_w0 = 0; s_w1 = nw - 1; s_c0 = 0; s_c1 = last - base + 1; }
        __syncthreads();
        // the chunks that hold ranks r0 and r1 bound the part of the bitmap this unit needs
        if (!whole) {
            for (int c = tid; c < nch; c += DN_THREADS) {
                const int lo = cpre[c], hi = (c + 1 < nch) ? cpre[c + 1] : cnt;
                if (lo <= r0 && r0 < hi) s_ca = c;
                if (r1 < cnt && lo <= r1 && r1 < hi) s_cb = c;
            }
            __syncthreads();
        }
        const int ca = s_ca, cb = s_cb;
        for (int c = ca + warp; c <= cb; c += DN_WARPS) {
            const int w = (c << 5) + lane;
            const unsigned word = (w < nw) ? src[w] : 0u;
            const int pc = __popc(word);
            const int start = cpre[c] + warp_incl_scan(pc) - pc;       // rank of this word's first bit
            if (w < nw) {
                bm[w] = word;
                pre[w] = (short)max(-32768, min(32767, start - r0));
                if (start <= r0 && r0 < start + pc) { s_w0 = w; s_c0 = (w << 5) + nth_set_bit(word, r0 - start); }
                if (r1 < cnt && start <= r1 && r1 < start + pc) { s_w1 = w; s_c1 = (w << 5) + nth_set_bit(word, r1 - start); }
            }
        }
        __syncthreads();
        // the unit owns the columns base + [lo_rel, hi_rel)
        const unsigned lo_rel = (unsigned)s_c0, hi_rel = (unsigned)s_c1;
        const int c_lo_abs = base + (int)lo_rel, c_hi_abs = base + (int)hi_rel;
        const unsigned span_bits = (unsigned)nw * 32u;

        for (i64 e0 = ps; e0 < pe; e0 += DN_ENTRIES) {
            // ---- round, step 1: one lane per A entry finds the entry's B-row segment inside the
            // unit's column range; non-empty segments are appended to the item list
            if (tid == 0) { s_items = 0; s_fetch = 0; s_nlong = 0; s_sumlen = 0; }
            __syncthreads();
            const i64 e1 = min(pe, e0 + DN_ENTRIES);
            for (i64 p = e0 + tid; p < e1; p += DN_THREADS) {
                const int k = __ldg(A.crd + p);
                if ((unsigned)k >= (unsigned)B.nrows) continue;
                const i64 qs = __ldg(B.pos + k);
                const int len = (int)(__ldg(B.pos + k + 1) - qs);
                int s0 = 0, s1 = len;
                if (!whole && len > 0) {
                    const int* __restrict__ ck = B.crd + qs;
                    s0 = lane_lower_bound(ck, 0, len, c_lo_abs);
                    s1 = lane_lower_bound(ck, s0, len, c_hi_abs);
                }
                if (s1 > s0) {
                    const int i = atomicAdd(&s_items, 1);
                    item_q[i] = qs + s0;
                    item_len[i] = s1 - s0;
                    item_a[i] = __ldg(Aval + p);
                    atomicAdd(&s_sumlen, s1 - s0);
                    if (s1 - s0 >= DN_LONG) {
                        const int l = atomicAdd(&s_nlong, 1);
                        if (l < DN_LONG_CAP) { s_long[l] = i; item_len[i] = -(s1 - s0); }   // negative: taken by the CTA-wide pass
                    }
                }
            }
            __syncthreads();
            // ---- step 2: lane groups pull items; group size ~ mean segment length
            const int n_items = s_items;
            int gs = 32;
            {
                const float avg = (float)s_sumlen / fmaxf(1.0f, (float)n_items);
                while (gs > 1 && (float)(gs >> 1) >= avg) gs >>= 1;
            }
            const int lg = __ffs(gs) - 1;
            const int gl = tid & (gs - 1);
            const unsigned gshift = (unsigned)(lane - gl);
            const unsigned gmask = (gs == 32) ? 0xffffffffu : (((1u << gs) - 1u) << gshift);
            const int batch = gs >= 8 ? 1 : (8 >> lg);          // items a group takes per fetch
            for (;;) {
                int i0 = 0;
                if (gl == 0) i0 = atomicAdd(&s_fetch, batch);
                i0 = __shfl_sync(gmask, i0, (int)gshift);
                if (i0 >= n_items) break;
                const int i1 = min(n_items, i0 + batch);
                for (int i = i0; i < i1; ++i) {
                    const int len = item_len[i];
                    if (len < 0) continue;
                    const int* __restrict__ ck = B.crd + item_q[i];
                    const T* __restrict__ vk = Bval + item_q[i];
                    const T a = item_a[i];
                    int t = gl;
                    for (; t + gs < len; t += 2 * gs) {         // two products in flight per lane
                        const unsigned rel0 = (unsigned)(__ldg(ck + t) - base);
                        const unsigned rel1 = (unsigned)(__ldg(ck + t + gs) - base);
                        const T v0 = __ldg(vk + t), v1 = __ldg(vk + t + gs);
                        if (rel0 < span_bits) {
                            const int slot = pre[rel0 >> 5] + __popc(bm[rel0 >> 5] & ((1u << (rel0 & 31)) - 1u));
                            if ((unsigned)slot < (unsigned)CAP) atomicAdd(&acc[slot], a * v0);
                        }
                        if (rel1 < span_bits) {
                            const int slot = pre[rel1 >> 5] + __popc(bm[rel1 >> 5] & ((1u << (rel1 & 31)) - 1u));
                            if ((unsigned)slot < (unsigned)CAP) atomicAdd(&acc[slot], a * v1);
                        }
                    }
                    if (t < len) {
                        const unsigned rel0 = (unsigned)(__ldg(ck + t) - base);
                        if (rel0 < span_bits) {
                            const int slot = pre[rel0 >> 5] + __popc(bm[rel0 >> 5] & ((1u << (rel0 & 31)) - 1u));
                            if ((unsigned)slot < (unsigned)CAP) atomicAdd(&acc[slot], a * __ldg(vk + t));
                        }
                    }
                }
            }
            // ---- step 3: very long segments, all threads of the CTA together
            const int n_long = min(s_nlong, DN_LONG_CAP);
            for (int l = 0; l < n_long; ++l) {
                const int i = s_long[l];
                const int len = -item_len[i];
                const int* __restrict__ ck = B.crd + item_q[i];
                const T* __restrict__ vk = Bval + item_q[i];
                const T a = item_a[i];
                for (int t = tid; t < len; t += DN_THREADS) {
                    const unsigned rel0 = (unsigned)(__ldg(ck + t) - base);
                    if (rel0 < span_bits) {
                        const int slot = pre[rel0 >> 5] + __popc(bm[rel0 >> 5] & ((1u << (rel0 & 31)) - 1u));
                        if ((unsigned)slot < (unsigned)CAP) atomicAdd(&acc[slot], a * __ldg(vk + t));
                    }
                }
            }
            __syncthreads();
        }

        // copy out: values are already in output order.  The coordinates are expanded from the
        // bitmap into shared memory (the accumulator's storage, once the values have left) so
        // that the global stores are contiguous.
        const i64 o0 = out0 + r0;
        for (int x = tid; x < nout; x += DN_THREADS) Cval[o0 + x] = acc[x];
        __syncthreads();
        int* stage = reinterpret_cast<int*>(acc);
        const int w_first = s_w0, w_last = s_w1;
        for (int w = w_first + tid; w <= w_last; w += DN_THREADS) {
            unsigned word = bm[w];
            int slot = pre[w];
            if (w == w_first) {                         // drop the bits below the unit's first column
                const unsigned below = (1u << (lo_rel & 31)) - 1u;
                slot += __popc(word & below);
                word &= ~below;
            }
            if (w == w_last && (hi_rel >> 5) == (unsigned)w) word &= (1u << (hi_rel & 31)) - 1u;
            const int col0 = base + (w << 5);
            while (word) {
                const int b = __ffs(word) - 1;
                word &= word - 1;
                if ((unsigned)slot < (unsigned)nout) stage[slot] = col0 + b;
                ++slot;
            }
        }
        __syncthreads();
        for (int x = tid; x < nout; x += DN_THREADS) Ccrd[o0 + x] = stage[x];
        __syncthreads();
        for (int x = tid; x < nout; x += DN_THREADS) acc[x] = 0;
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
    dense_sym_cta_kernel<<<persistent_grid(c, per_sm, -1), DC_THREADS, smem, c.stream>>>(c.ctl, c.dense_smem_words, A, B, c.tab);
    ++c.launches;
    return cudaGetLastError();
}

template <typename T>
static cudaError_t num_warp_t(const LaunchCtx& c, int n_host, const Csr& A, const Csr& B, const i64* rowptr, int* Ccrd, void* Cval) {
    int per_sm = 0;
    const size_t smem = (size_t)DW_WARPS * (sizeof(T) * DENSE_WARP_ACC + 6 * (size_t)DENSE_WARP_BM_WORDS);
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(dense_num_warp_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, dense_num_warp_kernel<T>, DW_THREADS, smem)) != cudaSuccess) return e;
    const i64 work = n_host >= 0 ? ((i64)n_host + DW_WARPS - 1) / DW_WARPS : -1;
    dense_num_warp_kernel<T><<<persistent_grid(c, per_sm, work), DW_THREADS, smem, c.stream>>>(c.ctl, A, B, c.tab, rowptr, Ccrd, (T*)Cval);
    ++c.launches;
    return cudaGetLastError();
}

cudaError_t launch_dense_num_warp(const LaunchCtx& c, int n_host, const Csr& A, const Csr& B,
                                  const i64* rowptr, int* Ccrd, void* Cval) {
    return c.is_f64 ? num_warp_t<double>(c, n_host, A, B, rowptr, Ccrd, Cval)
                    : num_warp_t<float>(c, n_host, A, B, rowptr, Ccrd, Cval);
}

template <typename T>
static cudaError_t num_cta_t(const LaunchCtx& c, int n_units_host, int words, const Csr& A, const Csr& B,
                             const i64* rowptr, int* Ccrd, void* Cval) {
    const int CAP = c.prm.unit_outputs;
    const size_t smem = sizeof(T) * (size_t)CAP + (sizeof(T) + 12) * (size_t)DN_ENTRIES + (size_t)words * 4 + (size_t)words * 2 + 16;
    cudaError_t e;
    int per_sm = 0;
    auto k = dense_num_cta_kernel<T>;
    if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, DN_THREADS, smem)) != cudaSuccess) return e;
    k<<<persistent_grid(c, per_sm, n_units_host), DN_THREADS, smem, c.stream>>>(c.ctl, words, CAP, A, B, c.tab, rowptr, Ccrd, (T*)Cval);
    ++c.launches;
    return cudaGetLastError();
}

cudaError_t launch_dense_num_cta(const LaunchCtx& c, int n_units_host, int max_span_words, const Csr& A, const Csr& B,
                                 const i64* rowptr, int* Ccrd, void* Cval) {
    int words = max_span_words > 0 ? max_span_words : c.dense_smem_words;
    words = (words + 31) & ~31;
    return c.is_f64 ? num_cta_t<double>(c, n_units_host, words, A, B, rowptr, Ccrd, Cval)
                    : num_cta_t<float>(c, n_units_host, words, A, B, rowptr, Ccrd, Cval);
}

}  // namespace spws
