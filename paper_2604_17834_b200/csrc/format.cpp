// Host-side format construction (Sec. 2.3 "Sparse Formats", Sec. 3.3 task split).
#include "format.h"

#include <algorithm>
#include <climits>
#include <cstring>
#include <numeric>
#include <queue>
#include <utility>

#include "kernels.h"
#include "spmm_b200.h"

namespace spmm {

static inline int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }

int validate_csr(const CsrView& a) {
    if (a.m < 0 || a.k < 0 || !a.row_ptr) return SPMM_ERR_INVALID_ARG;
    if (a.row_ptr[0] != 0) return SPMM_ERR_INVALID_ARG;
    for (int64_t i = 0; i < a.m; ++i)
        if (a.row_ptr[i + 1] < a.row_ptr[i]) return SPMM_ERR_INVALID_ARG;
    if (a.row_ptr[a.m] != a.nnz) return SPMM_ERR_INVALID_ARG;
    if (a.nnz > 0 && (!a.col_idx || !a.vals)) return SPMM_ERR_INVALID_ARG;
    for (int64_t i = 0; i < a.m; ++i) {
        int64_t prev = -1;
        for (int64_t p = a.row_ptr[i]; p < a.row_ptr[i + 1]; ++p) {
            const int64_t c = a.col_idx[p];
            if (c < 0 || c >= a.k) return SPMM_ERR_OUT_OF_RANGE;
            if (c <= prev) return SPMM_ERR_UNSORTED;
            prev = c;
        }
    }
    return SPMM_OK;
}

int coo_to_csr(int64_t m, int64_t k, int64_t nnz, const int32_t* rows, const int32_t* cols,
               const uint8_t* vals, int es, CsrOwned* out) {
    if (m < 0 || k < 0 || nnz < 0) return SPMM_ERR_INVALID_ARG;
    if (nnz > 0 && (!rows || !cols || !vals)) return SPMM_ERR_INVALID_ARG;
    for (int64_t p = 0; p < nnz; ++p)
        if (rows[p] < 0 || rows[p] >= m || cols[p] < 0 || cols[p] >= k) return SPMM_ERR_OUT_OF_RANGE;
    std::vector<int64_t> perm(static_cast<size_t>(nnz));
    std::iota(perm.begin(), perm.end(), int64_t{0});
    std::stable_sort(perm.begin(), perm.end(), [&](int64_t x, int64_t y) {
        if (rows[x] != rows[y]) return rows[x] < rows[y];
        return cols[x] < cols[y];
    });
    for (int64_t p = 1; p < nnz; ++p)
        if (rows[perm[p]] == rows[perm[p - 1]] && cols[perm[p]] == cols[perm[p - 1]])
            return SPMM_ERR_UNSORTED;
    out->row_ptr.assign(static_cast<size_t>(m) + 1, 0);
    out->col_idx.resize(static_cast<size_t>(nnz));
    out->vals.resize(static_cast<size_t>(nnz) * es);
    for (int64_t p = 0; p < nnz; ++p) {
        const int64_t s = perm[p];
        out->row_ptr[static_cast<size_t>(rows[s]) + 1]++;
        out->col_idx[p] = cols[s];
        std::memcpy(&out->vals[static_cast<size_t>(p) * es], vals + static_cast<size_t>(s) * es, es);
    }
    for (int64_t i = 0; i < m; ++i) out->row_ptr[i + 1] += out->row_ptr[i];
    return SPMM_OK;
}

// ----------------------------------------------------------------------------- BCSR

int build_bcsr(const CsrView& a, int b, BcsrHost* out) {
    if (b != 16 && b != 32 && b != 64 && b != 128) return SPMM_ERR_UNSUPPORTED;
    out->b = b;
    const int64_t nbr = cdiv(a.m, b), nbc = cdiv(a.k, b);
    out->nbr = nbr;
    out->nbc = nbc;
    out->block_row_ptr.assign(static_cast<size_t>(nbr) + 1, 0);
    out->block_col_idx.clear();

    // pass 1: which block columns each block-row touches (structural: any stored entry)
    std::vector<int64_t> stamp(static_cast<size_t>(nbc), -1);
    std::vector<int32_t> found;
    for (int64_t I = 0; I < nbr; ++I) {
        found.clear();
        const int64_t r1 = std::min<int64_t>(a.m, (I + 1) * b);
        for (int64_t i = I * b; i < r1; ++i)
            for (int64_t p = a.row_ptr[i]; p < a.row_ptr[i + 1]; ++p) {
                const int64_t J = a.col_idx[p] / b;
                if (stamp[J] != I) {
                    stamp[J] = I;
                    found.push_back(static_cast<int32_t>(J));
                }
            }
        std::sort(found.begin(), found.end());
        out->block_col_idx.insert(out->block_col_idx.end(), found.begin(), found.end());
        if (out->block_col_idx.size() >= (size_t{1} << 31)) return SPMM_ERR_TOO_LARGE;
        out->block_row_ptr[I + 1] = static_cast<int32_t>(out->block_col_idx.size());
    }
    const int64_t nnzb = static_cast<int64_t>(out->block_col_idx.size());
    out->nnzb = nnzb;

    // pass 2: scatter the values into their dense tiles
    const size_t tile_bytes = static_cast<size_t>(b) * b * a.es;
    out->blocks.assign(static_cast<size_t>(nnzb) * tile_bytes, 0);
    std::vector<int32_t> slot_of(static_cast<size_t>(nbc), -1);
    for (int64_t I = 0; I < nbr; ++I) {
        for (int32_t p = out->block_row_ptr[I]; p < out->block_row_ptr[I + 1]; ++p)
            slot_of[out->block_col_idx[p]] = p;
        const int64_t r1 = std::min<int64_t>(a.m, (I + 1) * b);
        for (int64_t i = I * b; i < r1; ++i)
            for (int64_t p = a.row_ptr[i]; p < a.row_ptr[i + 1]; ++p) {
                const int64_t c = a.col_idx[p];
                const size_t dst = static_cast<size_t>(slot_of[c / b]) * tile_bytes +
                                   (static_cast<size_t>(i - I * b) * b + static_cast<size_t>(c % b)) * a.es;
                std::memcpy(&out->blocks[dst], a.vals + static_cast<size_t>(p) * a.es, a.es);
            }
    }

    finish_bcsr_host(out);      // row order (most stored blocks first, ties by index), empty rows, distinct columns
    return SPMM_OK;
}

int build_tile_schedule(const std::vector<int32_t>& units, const std::vector<int32_t>& lens, int fixed_cost, int n_tt,
                        int slab_w, int n_ctas, BcsrSchedule* out, int64_t unit_cost, const std::vector<int64_t>* initial,
                        std::vector<int64_t>* final_loads) {
    if (n_tt <= 0 || slab_w <= 0 || n_ctas <= 0 || units.size() != lens.size()) return SPMM_ERR_INVALID_ARG;
    if (initial && initial->size() != static_cast<size_t>(n_ctas)) return SPMM_ERR_INVALID_ARG;
    out->n_tt = n_tt;
    out->slab_w = slab_w;
    out->n_ctas = n_ctas;
    const int64_t nu = static_cast<int64_t>(units.size());
    const int64_t ntiles = nu * n_tt;
    if (ntiles >= (int64_t{1} << 30)) return SPMM_ERR_TOO_LARGE;
    using Load = std::pair<int64_t, int32_t>;   // (load, CTA): smallest load, then lowest CTA, on top
    std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
    for (int32_t c = 0; c < n_ctas; ++c) heap.push(Load(initial ? (*initial)[c] : 0, c));
    std::vector<int32_t> owner(static_cast<size_t>(ntiles));
    std::vector<int32_t> seq_I(static_cast<size_t>(ntiles)), seq_t(static_cast<size_t>(ntiles));
    std::vector<int32_t> count(static_cast<size_t>(n_ctas), 0);
    int64_t n = 0;
    for (int t0 = 0; t0 < n_tt; t0 += slab_w) {
        const int t1 = std::min(n_tt, t0 + slab_w);
        for (int64_t r = 0; r < nu; ++r) {
            const int32_t I = units[r];
            const int64_t cost = (lens[r] + fixed_cost) * unit_cost;
            for (int t = t0; t < t1; ++t, ++n) {
                Load top = heap.top();
                heap.pop();
                owner[n] = top.second;
                seq_I[n] = I;
                seq_t[n] = t;
                count[top.second]++;
                top.first += cost;
                heap.push(top);
            }
        }
    }
    out->cta_ptr.assign(static_cast<size_t>(n_ctas) + 1, 0);
    for (int c = 0; c < n_ctas; ++c) out->cta_ptr[c + 1] = out->cta_ptr[c] + count[c];
    out->tiles.assign(static_cast<size_t>(2 * ntiles), 0);
    std::vector<int32_t> pos(out->cta_ptr.begin(), out->cta_ptr.end() - 1);
    for (int64_t i = 0; i < ntiles; ++i) {
        const int32_t dst = pos[owner[i]]++;
        out->tiles[2 * dst] = seq_I[i];
        out->tiles[2 * dst + 1] = seq_t[i];
    }
    if (final_loads) {
        final_loads->assign(static_cast<size_t>(n_ctas), 0);
        while (!heap.empty()) {
            (*final_loads)[heap.top().second] = heap.top().first;
            heap.pop();
        }
    }
    return SPMM_OK;
}

int build_bcsr_schedule(const BcsrHost& f, int n_tt, int slab_w, int n_ctas, BcsrSchedule* out) {
    std::vector<int32_t> lens(static_cast<size_t>(f.nbr));
    for (int64_t r = 0; r < f.nbr; ++r) {
        const int32_t I = f.row_order[r];
        lens[r] = f.block_row_ptr[I + 1] - f.block_row_ptr[I];
    }
    return build_tile_schedule(f.row_order, lens, kTileFixedCost, n_tt, slab_w, n_ctas, out);
}

int build_bcsr_ksplit(const BcsrHost& f, int n_tt, int n_ctas, std::vector<int32_t>* units, int64_t* n_slots, int32_t* cap_out) {
    units->clear();
    *n_slots = 0;
    int64_t total = 0;
    int32_t longest = 0;
    for (int64_t I = 0; I < f.nbr; ++I) {
        const int32_t len = f.block_row_ptr[I + 1] - f.block_row_ptr[I];
        total += len + kTileFixedCost;
        longest = std::max(longest, len);
    }
    total *= n_tt;
    const int64_t quarter = (total + 4 * int64_t{n_ctas} - 1) / (4 * int64_t{n_ctas});
    const int32_t cap = static_cast<int32_t>(std::min<int64_t>(std::max<int64_t>(kKSplitMinCap, quarter), INT32_MAX));
    *cap_out = cap;
    if (longest <= cap) return SPMM_OK;
    // slots: split block-rows in ascending index, parts ascending
    std::vector<int32_t> first_slot(static_cast<size_t>(f.nbr), -1);
    int64_t slots = 0;
    for (int64_t I = 0; I < f.nbr; ++I) {
        const int32_t len = f.block_row_ptr[I + 1] - f.block_row_ptr[I];
        if (len > cap) {
            first_slot[I] = static_cast<int32_t>(slots);
            slots += (len + cap - 1) / cap;
        }
    }
    if (slots >= (int64_t{1} << 30)) return SPMM_ERR_TOO_LARGE;
    for (int64_t r = 0; r < f.nbr; ++r) {
        const int32_t I = f.row_order[r];
        const int32_t p0 = f.block_row_ptr[I];
        const int64_t len = f.block_row_ptr[I + 1] - p0;
        if (len <= cap) {
            units->insert(units->end(), {I, p0, static_cast<int32_t>(p0 + len), -1});
            continue;
        }
        const int64_t parts = (len + cap - 1) / cap;
        for (int64_t j = 0; j < parts; ++j)
            units->insert(units->end(), {I, static_cast<int32_t>(p0 + j * len / parts), static_cast<int32_t>(p0 + (j + 1) * len / parts),
                                         static_cast<int32_t>(first_slot[I] + j)});
    }
    *n_slots = slots;
    return SPMM_OK;
}

int build_bcsr_stack(const BcsrHost& f, int min_fill_pct, BcsrStack* out) {
    *out = BcsrStack();
    out->stacked.assign(static_cast<size_t>(f.nbr), 0);
    if (f.b >= 128 || min_fill_pct < 0) return SPMM_OK;
    const int R = 128 / f.b;
    out->R = R;
    out->min_fill_pct = min_fill_pct > 0 ? min_fill_pct : bcsr_stack_default_fill(f.b);
    out->ptr.push_back(0);
    std::vector<int32_t> cursor(static_cast<size_t>(R));
    // block-rows per block column (ascending), position of every block-row in row_order
    std::vector<int64_t> col_ptr(static_cast<size_t>(f.nbc) + 1, 0);
    for (int64_t q = 0; q < f.nnzb; ++q) ++col_ptr[f.block_col_idx[q] + 1];
    for (int64_t J = 0; J < f.nbc; ++J) col_ptr[J + 1] += col_ptr[J];
    std::vector<int32_t> col_rows(static_cast<size_t>(f.nnzb));
    {
        std::vector<int64_t> fill(col_ptr.begin(), col_ptr.end() - 1);
        for (int64_t I = 0; I < f.nbr; ++I)
            for (int32_t q = f.block_row_ptr[I]; q < f.block_row_ptr[I + 1]; ++q) col_rows[fill[f.block_col_idx[q]]++] = static_cast<int32_t>(I);
    }
    std::vector<int32_t> pos(static_cast<size_t>(f.nbr));
    std::vector<uint8_t> is_free(static_cast<size_t>(f.nbr));
    for (int64_t r = 0; r < f.nbr; ++r) {
        pos[f.row_order[r]] = static_cast<int32_t>(r);
        is_free[r] = f.block_row_ptr[r + 1] > f.block_row_ptr[r];
    }
    std::vector<int32_t> shared(static_cast<size_t>(f.nbr), 0), touched, rows(static_cast<size_t>(R));
    int64_t work = 0;
    for (int64_t r0 = 0; r0 < f.nbr; ++r0) {
        const int32_t seed = f.row_order[r0];
        if (f.block_row_ptr[seed + 1] == f.block_row_ptr[seed]) break;      // row_order lists empty block-rows last
        if (!is_free[seed]) continue;
        int64_t w = 0;
        for (int32_t q = f.block_row_ptr[seed]; q < f.block_row_ptr[seed + 1]; ++q)
            w += col_ptr[f.block_col_idx[q] + 1] - col_ptr[f.block_col_idx[q]];
        if (work + w > kBcsrGroupWorkLimit) break;
        work += w;
        // block columns shared with the seed, per free block-row
        touched.clear();
        for (int32_t q = f.block_row_ptr[seed]; q < f.block_row_ptr[seed + 1]; ++q) {
            const int32_t J = f.block_col_idx[q];
            for (int64_t t = col_ptr[J]; t < col_ptr[J + 1]; ++t) {
                const int32_t r = col_rows[t];
                if (r == seed || !is_free[r]) continue;
                if (shared[r]++ == 0) touched.push_back(r);
            }
        }
        const bool enough = static_cast<int64_t>(touched.size()) >= R - 1;
        if (enough)
            std::partial_sort(touched.begin(), touched.begin() + (R - 1), touched.end(), [&](int32_t x, int32_t y) {
                return shared[x] != shared[y] ? shared[x] > shared[y] : pos[x] < pos[y];
            });
        rows[0] = seed;
        for (int i = 1; enough && i < R; ++i) rows[i] = touched[i - 1];
        for (int32_t r : touched) shared[r] = 0;
        if (!enough) continue;
        std::sort(rows.begin(), rows.end(), [&](int32_t x, int32_t y) { return pos[x] < pos[y]; });
        int64_t stored = 0;
        for (int i = 0; i < R; ++i) {
            cursor[i] = f.block_row_ptr[rows[i]];
            stored += f.block_row_ptr[rows[i] + 1] - f.block_row_ptr[rows[i]];
        }
        // merge of the R ascending column lists
        const size_t col0 = out->col_idx.size();
        for (;;) {
            int32_t J = INT32_MAX;
            for (int i = 0; i < R; ++i)
                if (cursor[i] < f.block_row_ptr[rows[i] + 1]) J = std::min(J, f.block_col_idx[cursor[i]]);
            if (J == INT32_MAX) break;
            out->col_idx.push_back(J);
            for (int i = 0; i < R; ++i) {
                if (cursor[i] < f.block_row_ptr[rows[i] + 1] && f.block_col_idx[cursor[i]] == J) out->src.push_back(cursor[i]++);
                else out->src.push_back(-1);
            }
        }
        const int64_t U = static_cast<int64_t>(out->col_idx.size() - col0);
        if (100 * stored >= static_cast<int64_t>(out->min_fill_pct) * R * U) {
            for (int i = 0; i < R; ++i) {
                out->rows.push_back(rows[i]);
                out->stacked[rows[i]] = 1;
                is_free[rows[i]] = 0;
            }
            out->ptr.push_back(static_cast<int32_t>(out->col_idx.size()));
        } else {
            out->col_idx.resize(col0);
            out->src.resize(col0 * R);
        }
    }
    out->ng = static_cast<int64_t>(out->ptr.size()) - 1;
    out->ns = static_cast<int64_t>(out->col_idx.size());
    if (out->ns * 128 >= (int64_t{1} << 31)) {     // row coordinate of the stacked values' tensor map
        const int keepR = out->R, keepF = out->min_fill_pct;
        *out = BcsrStack();
        out->R = keepR;
        out->min_fill_pct = keepF;
        out->stacked.assign(static_cast<size_t>(f.nbr), 0);
        out->ptr.push_back(0);
    }
    return SPMM_OK;
}

// ----------------------------------------------------------------------------- WCSR

int build_wcsr(const CsrView& a, int wh, int b_col, int T, int n_bins, WcsrHost* out) {
    if (wh != 16 && wh != 64) return SPMM_ERR_UNSUPPORTED;
    if (b_col * a.es != 32) return SPMM_ERR_UNSUPPORTED;
    if (T < 0 || T % b_col != 0 || n_bins <= 0) return SPMM_ERR_INVALID_ARG;
    out->wh = wh;
    out->b_col = b_col;
    const int64_t nwin = cdiv(a.m, wh);
    out->nwin = nwin;
    out->window_row_ptr.assign(static_cast<size_t>(nwin) + 1, 0);
    out->window_col_idx.clear();

    // pass 1: per window, the ascending union of its rows' columns, padded with -1
    std::vector<int32_t> cols;
    std::vector<uint8_t> col_used(static_cast<size_t>(a.k), 0);
    int64_t P = 0;
    for (int64_t w = 0; w < nwin; ++w) {
        const int64_t r0 = w * wh, r1 = std::min<int64_t>(a.m, r0 + wh);
        cols.assign(a.col_idx + a.row_ptr[r0], a.col_idx + a.row_ptr[r1]);
        std::sort(cols.begin(), cols.end());
        cols.erase(std::unique(cols.begin(), cols.end()), cols.end());
        const int64_t len = cdiv(static_cast<int64_t>(cols.size()), b_col) * b_col;
        if (P + len >= (int64_t{1} << 31)) return SPMM_ERR_TOO_LARGE;
        for (int32_t c : cols) col_used[c] = 1;
        out->window_col_idx.insert(out->window_col_idx.end(), cols.begin(), cols.end());
        out->window_col_idx.insert(out->window_col_idx.end(), static_cast<size_t>(len) - cols.size(), -1);
        P += len;
        out->window_row_ptr[w + 1] = static_cast<int32_t>(P);
    }
    out->P = P;
    out->distinct_cols = std::count(col_used.begin(), col_used.end(), uint8_t{1});

    // pass 2: values, straight into the packed device layout
    out->packed.assign(static_cast<size_t>(P) * wh * a.es, 0);
    for (int64_t w = 0; w < nwin; ++w) {
        const int64_t r0 = w * wh, r1 = std::min<int64_t>(a.m, r0 + wh);
        const int32_t* wc = out->window_col_idx.data() + out->window_row_ptr[w];
        const int64_t base = out->window_row_ptr[w];
        for (int64_t i = r0; i < r1; ++i) {
            int64_t q = 0;   // both lists ascend: walk them together
            for (int64_t p = a.row_ptr[i]; p < a.row_ptr[i + 1]; ++p) {
                const int32_t c = a.col_idx[p];
                while (wc[q] != c) ++q;
                std::memcpy(&out->packed[wcsr_packed_offset(wh, b_col, a.es, static_cast<int>(i - r0), base + q)],
                            a.vals + static_cast<size_t>(p) * a.es, a.es);
            }
        }
    }

    wcsr_reuse_classes(out->window_col_idx.data(), P, a.k, &out->grp_class);
    return plan_wcsr(out, T, n_bins, a.es);
}

void wcsr_reuse_classes(const int32_t* window_col_idx, int64_t P, int64_t k, std::vector<uint8_t>* grp_class) {
    // gathers per B row = windows whose column list holds it
    std::vector<int32_t> refs(static_cast<size_t>(k), 0);
    for (int64_t q = 0; q < P; ++q)
        if (window_col_idx[q] >= 0) refs[window_col_idx[q]]++;
    // rows gathered more than once, most gathered first (ties: lower index first)
    std::vector<int32_t> order;
    for (int64_t c = 0; c < k; ++c)
        if (refs[c] > 1) order.push_back(static_cast<int32_t>(c));
    std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) { return refs[x] > refs[y]; });
    std::vector<uint8_t> cls(static_cast<size_t>(k), 0);
    for (size_t r = 0; r < order.size(); ++r) {
        int level = 7;
        for (size_t lim = kWcsrTopClassRows; level > 0 && r >= lim; lim *= 2) --level;
        if (level == 0) break;
        cls[order[r]] = static_cast<uint8_t>(level);
    }
    grp_class->assign(static_cast<size_t>(P / 4), 0);
    for (int64_t q = 0; q < P; ++q)
        if (window_col_idx[q] >= 0) {
            uint8_t& g = (*grp_class)[static_cast<size_t>(q >> 2)];
            g = std::max(g, cls[window_col_idx[q]]);
        }
}

// Largest bin load of the longest-processing-time assignment when windows are cut into chunks of T.
static int64_t lpt_max_load(const std::vector<int32_t>& window_row_ptr, int64_t nwin, int T, int n_bins) {
    std::vector<int32_t> counts;
    for (int64_t w = 0; w < nwin; ++w) {
        int32_t len = window_row_ptr[w + 1] - window_row_ptr[w];
        for (; len > T; len -= T) counts.push_back(T);
        if (len > 0) counts.push_back(len);
    }
    std::sort(counts.begin(), counts.end(), std::greater<int32_t>());
    std::priority_queue<int64_t, std::vector<int64_t>, std::greater<int64_t>> heap;
    for (int j = 0; j < n_bins; ++j) heap.push(0);
    int64_t mx = 0;
    for (int32_t c : counts) {
        const int64_t l = heap.top() + c + kTaskFixedCost;
        heap.pop();
        heap.push(l);
        mx = std::max(mx, l);
    }
    return mx;
}

int default_split_cols(const std::vector<int32_t>& window_row_ptr, int64_t nwin, int64_t P, int n_bins) {
    // candidates: one bin's share of the padded columns and its half, quarter and eighth
    int cand[4];
    int64_t load[4], best = INT64_MAX;
    for (int i = 0; i < 4; ++i) {
        const int64_t t = ((P / n_bins) >> i) / 64 * 64;
        cand[i] = static_cast<int>(std::min<int64_t>(65536, std::max<int64_t>(128, t)));
        load[i] = (i > 0 && cand[i] == cand[i - 1]) ? load[i - 1] : lpt_max_load(window_row_ptr, nwin, cand[i], n_bins);
        best = std::min(best, load[i]);
    }
    for (int i = 0; i < 4; ++i)
        if (load[i] * 100 <= best * 102) return cand[i];
    return cand[3];
}

int plan_wcsr(WcsrHost* out, int T, int n_bins, int es) {
    const int64_t nwin = out->nwin, P = out->P;
    if (T == 0) T = default_split_cols(out->window_row_ptr, nwin, P, n_bins);
    out->T = T;

    // split plan: consecutive chunks of T columns; a window with one chunk writes C itself
    out->tasks.clear();
    out->merge_window.clear();
    out->merge_first.clear();
    out->merge_nparts.clear();
    out->n_empty = out->n_split = out->n_slots = 0;
    std::vector<int32_t> empty_windows;
    for (int64_t w = 0; w < nwin; ++w) {
        const int32_t len = out->window_row_ptr[w + 1] - out->window_row_ptr[w];
        if (len == 0) {
            empty_windows.push_back(static_cast<int32_t>(w));
            continue;
        }
        const int32_t nchunk = static_cast<int32_t>(cdiv(len, T));
        if (nchunk > 1) {
            out->merge_window.push_back(static_cast<int32_t>(w));
            out->merge_first.push_back(static_cast<int32_t>(out->n_slots));
            out->merge_nparts.push_back(nchunk);
            out->n_split++;
        }
        for (int32_t c = 0; c < nchunk; ++c) {
            WcsrTask t;
            t.window = static_cast<int32_t>(w);
            t.q0 = c * T;
            t.count = std::min(T, len - c * T);
            t.slot = nchunk > 1 ? static_cast<int32_t>(out->n_slots++) : -1;
            out->tasks.push_back(t);
        }
    }
    out->n_empty = static_cast<int64_t>(empty_windows.size());
    for (int32_t w : empty_windows) {
        out->merge_window.push_back(w);
        out->merge_first.push_back(-1);
        out->merge_nparts.push_back(0);
    }

    // bins: longest-processing-time assignment of tasks
    const int64_t ntasks = static_cast<int64_t>(out->tasks.size());
    std::vector<int32_t> order(static_cast<size_t>(ntasks));
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(),
                     [&](int32_t x, int32_t y) { return out->tasks[x].count > out->tasks[y].count; });
    using Load = std::pair<int64_t, int32_t>;   // (load, bin): smallest load, then lowest bin, on top
    std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
    for (int32_t bsel = 0; bsel < n_bins; ++bsel) heap.push(Load(0, bsel));
    std::vector<int32_t> bin_of(static_cast<size_t>(ntasks));
    std::vector<int32_t> bin_count(static_cast<size_t>(n_bins), 0);
    for (int32_t t : order) {
        Load top = heap.top();
        heap.pop();
        bin_of[t] = top.second;
        bin_count[top.second]++;
        top.first += out->tasks[t].count + kTaskFixedCost;
        heap.push(top);
    }
    out->bin_ptr.assign(static_cast<size_t>(n_bins) + 1, 0);
    for (int j = 0; j < n_bins; ++j) out->bin_ptr[j + 1] = out->bin_ptr[j] + bin_count[j];
    out->bin_tasks.assign(static_cast<size_t>(ntasks), 0);
    {
        std::vector<int32_t> fillpos(out->bin_ptr.begin(), out->bin_ptr.end() - 1);
        for (int64_t t = 0; t < ntasks; ++t) out->bin_tasks[fillpos[bin_of[t]]++] = static_cast<int32_t>(t);
    }

    // pipeline schedule: one fill per stage-sized run of columns (16 KB of gathered B rows at
    // 128 tokens: 64 columns of a 2-byte type, 32 of a 4-byte type), bin-major
    out->kt = wcsr_stage_cols(es);
    auto cut = [&](int kt, std::vector<int32_t>* fills, std::vector<int32_t>* bin_fill) -> int {
        fills->clear();
        bin_fill->assign(static_cast<size_t>(n_bins) + 1, 0);
        for (int j = 0; j < n_bins; ++j) {
            for (int32_t i = out->bin_ptr[j]; i < out->bin_ptr[j + 1]; ++i) {
                const WcsrTask& tk = out->tasks[out->bin_tasks[i]];
                const int32_t base = out->window_row_ptr[tk.window] + tk.q0;
                for (int32_t done = 0; done < tk.count; done += kt) {
                    const int32_t cnt = std::min(kt, tk.count - done);
                    const int32_t first = done == 0, last = done + kt >= tk.count;
                    fills->push_back(base + done);
                    fills->push_back(cnt | (first << 16) | (last << 17));
                }
            }
            if (fills->size() / 2 >= (size_t{1} << 31)) return SPMM_ERR_TOO_LARGE;
            (*bin_fill)[j + 1] = static_cast<int32_t>(fills->size() / 2);
        }
        return SPMM_OK;
    };
    int rc = cut(out->kt, &out->fills, &out->bin_fill);
    out->fills_narrow.clear();
    out->bin_fill_narrow.clear();
    if (!rc && es == 2 && out->wh == 16) rc = cut(kWcsrNarrowCols, &out->fills_narrow, &out->bin_fill_narrow);
    if (rc) return rc;
    return SPMM_OK;
}

}  // namespace spmm
