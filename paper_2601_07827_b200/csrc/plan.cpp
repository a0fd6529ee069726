// Planner implementation; see plan.h.
#include "plan.h"

#include <algorithm>
#include <cstdlib>
#include <sstream>

namespace btc {

size_t dtype_size(btc_dtype_t t)
{
    switch (t) {
    case BTC_F32: return 4;
    case BTC_F64: return 8;
    case BTC_C32: return 8;
    case BTC_C64: return 16;
    }
    return 0;
}

bool dtype_is_complex(btc_dtype_t t) { return t == BTC_C32 || t == BTC_C64; }

namespace {

inline int64_t iabs(int64_t x) { return x < 0 ? -x : x; }

struct LabelRow {
    int64_t label = 0, extent = 0;
    int64_t sA = 0, sB = 0, sD = 0;
    bool inA = false, inB = false, inD = false;
};

int find_label(const std::vector<LabelRow> &rows, int64_t label)
{
    for (size_t i = 0; i < rows.size(); ++i)
        if (rows[i].label == label) return int(i);
    return -1;
}

// Sufficient test that no two index tuples of D address the same element: with the modes of
// extent > 1 sorted by |stride|, every stride must exceed the span of all smaller ones.
bool d_may_alias(const TensorDesc &D)
{
    std::vector<std::pair<int64_t, int64_t>> se;
    for (size_t i = 0; i < D.extent.size(); ++i)
        if (D.extent[i] > 1) {
            if (D.stride[i] == 0) return true;
            se.emplace_back(iabs(D.stride[i]), D.extent[i]);
        }
    std::sort(se.begin(), se.end());
    int64_t span = 0;
    for (auto &p : se) {
        if (p.first < 1 + span) return true;
        span += p.first * (p.second - 1);
    }
    return false;
}

// Merge loop dimensions whose strides chain in every tensor: y follows x when
// stride_y == stride_x * extent_x for A, B and D alike.
void fuse_modes(std::vector<Mode> &g)
{
    bool changed = true;
    while (changed) {
        changed = false;
        for (size_t x = 0; x < g.size() && !changed; ++x)
            for (size_t y = 0; y < g.size() && !changed; ++y) {
                if (x == y) continue;
                if (g[y].sA == g[x].sA * g[x].extent && g[y].sB == g[x].sB * g[x].extent &&
                    g[y].sD == g[x].sD * g[x].extent) {
                    g[x].extent *= g[y].extent;
                    g.erase(g.begin() + y);
                    changed = true;
                }
            }
    }
}

int64_t product(const std::vector<Mode> &g)
{
    int64_t p = 1;
    for (auto &m : g) p *= m.extent;
    return p;
}

// offsets of all index tuples of `g`, first mode fastest
template <typename F>
std::vector<int64_t> build_table(const std::vector<Mode> &g, F stride_of)
{
    std::vector<int64_t> t(1, 0);
    for (auto &md : g) {
        const int64_t s = stride_of(md);
        const size_t len = t.size();
        t.resize(len * size_t(md.extent));
        for (int64_t i = 1; i < md.extent; ++i)
            for (size_t j = 0; j < len; ++j) t[size_t(i) * len + j] = t[j] + i * s;
    }
    return t;
}

void span_of(const TensorDesc &t, int64_t &lo, int64_t &hi)
{
    lo = hi = 0;
    for (size_t i = 0; i < t.extent.size(); ++i) {
        const int64_t d = t.stride[i] * (t.extent[i] - 1);
        if (d < 0) lo += d; else hi += d;
    }
}

// Split mode `idx` of `g` into an inner part of extent f (a divisor of its extent, f > 1) that
// stays at `idx`, and an outer part appended at the end.
void split_mode(std::vector<Mode> &g, size_t idx, int64_t f)
{
    Mode outer = g[idx];
    outer.extent = g[idx].extent / f;
    outer.sA = g[idx].sA * f;
    outer.sB = g[idx].sB * f;
    outer.sD = g[idx].sD * f;
    g[idx].extent = f;
    if (outer.extent > 1) g.push_back(outer);
}

int64_t largest_divisor_at_most(int64_t n, int64_t cap)
{
    for (int64_t f = std::min(n, cap); f >= 1; --f)
        if (n % f == 0) return f;
    return 1;
}

}  // namespace

int make_plan(const PlanRequest &req, Plan &plan)
{
    const TensorDesc *T[3] = {&req.A, &req.B, &req.D};
    const std::vector<int64_t> *L[3] = {&req.labelsA, &req.labelsB, &req.labelsD};

    // ---- checks (Sec. "Algorithm Structure"; test list items 26-28; Eq. (FreeD)) ----
    for (int t = 0; t < 3; ++t) {
        if (T[t]->extent.size() > BTC_MAX_RANK) return BTC_ERR_INVALID_ARGUMENT;
        if (T[t]->extent.size() != T[t]->stride.size() || T[t]->extent.size() != L[t]->size())
            return BTC_ERR_INVALID_ARGUMENT;
        for (int64_t e : T[t]->extent)
            if (e < 1) return BTC_ERR_INVALID_EXTENT;
    }
    // Element types (Sec. "Challenge: Datatypes"): the tensors may mix real and complex elements of one part
    // width; D must be complex when an input is.  Other mixes (32- with 64-bit parts) are not supported.
    const bool mixed = req.A.dtype != req.D.dtype || req.B.dtype != req.D.dtype || (req.has_c && req.C.dtype != req.D.dtype);
    {
        auto part = [](btc_dtype_t t) { return (t == BTC_F32 || t == BTC_C32) ? 4 : 8; };
        const btc_dtype_t c_type = req.has_c ? req.C.dtype : req.D.dtype;
        if (part(req.A.dtype) != part(req.D.dtype) || part(req.B.dtype) != part(req.D.dtype) || part(c_type) != part(req.D.dtype))
            return BTC_ERR_NOT_SUPPORTED;
        if (!dtype_is_complex(req.D.dtype) &&
            (dtype_is_complex(req.A.dtype) || dtype_is_complex(req.B.dtype) || dtype_is_complex(c_type)))
            return BTC_ERR_NOT_SUPPORTED;
    }
    for (size_t i = 0; i < req.labelsD.size(); ++i)
        for (size_t j = 0; j < i; ++j)
            if (req.labelsD[i] == req.labelsD[j]) return BTC_ERR_NOT_SUPPORTED;

    std::vector<LabelRow> rows;
    for (int t = 0; t < 3; ++t)
        for (size_t i = 0; i < L[t]->size(); ++i) {
            int k = find_label(rows, (*L[t])[i]);
            if (k < 0) {
                if (rows.size() == BTC_MAX_LABELS) return BTC_ERR_INVALID_ARGUMENT;
                LabelRow r;
                r.label = (*L[t])[i];
                r.extent = T[t]->extent[i];
                rows.push_back(r);
                k = int(rows.size()) - 1;
            } else if (rows[k].extent != T[t]->extent[i]) {
                return BTC_ERR_EXTENT_MISMATCH;
            }
            // a repeated label acts as one mode whose stride is the sum (Note 6)
            if (t == 0) { rows[k].sA += T[t]->stride[i]; rows[k].inA = true; }
            if (t == 1) { rows[k].sB += T[t]->stride[i]; rows[k].inB = true; }
            if (t == 2) { rows[k].sD += T[t]->stride[i]; rows[k].inD = true; }
        }
    for (auto &r : rows)
        if (r.inD && !r.inA && !r.inB) return BTC_ERR_LABEL_ONLY_IN_D;
    if (req.has_c) {
        if (req.C.extent.size() != req.D.extent.size() || req.labelsC.size() != req.labelsD.size())
            return BTC_ERR_C_D_MISMATCH;
        for (size_t i = 0; i < req.D.extent.size(); ++i)
            if (req.C.extent[i] != req.D.extent[i] || req.C.stride[i] != req.D.stride[i] ||
                req.labelsC[i] != req.labelsD[i])
                return BTC_ERR_C_D_MISMATCH;
    }
    if (d_may_alias(req.D)) return BTC_ERR_D_ALIASING;

    // ---- classify (Sec. "Operations": H, F_A, F_B, P; I_A / I_B of Case 4) ----
    plan = Plan();
    plan.dtype = req.D.dtype;
    plan.mixed = mixed;
    plan.cplxA = dtype_is_complex(req.A.dtype);
    plan.cplxB = dtype_is_complex(req.B.dtype);
    plan.cplxC = dtype_is_complex(req.has_c ? req.C.dtype : req.D.dtype);
    plan.conjA = req.conjA && plan.cplxA;
    plan.conjB = req.conjB && plan.cplxB;
    plan.conjC = req.conjC && plan.cplxC;
    plan.has_c_desc = req.has_c;
    for (auto &r : rows) {
        if (r.extent == 1) continue;  // contributes no loop and no offset
        Mode md;
        md.extent = r.extent;
        md.sA = r.sA; md.sB = r.sB; md.sD = r.sD;
        if (r.inA && r.inB && r.inD) plan.batch.push_back(md);
        else if (r.inA && r.inD) plan.m.push_back(md);
        else if (r.inB && r.inD) plan.n.push_back(md);
        else if (r.inA && r.inB) plan.k.push_back(md);
        else { plan.k.push_back(md); plan.has_isolated = true; }  // summed; stride 0 elsewhere
    }
    span_of(req.A, plan.spanA_lo, plan.spanA_hi);
    span_of(req.B, plan.spanB_lo, plan.spanB_hi);
    span_of(req.D, plan.spanD_lo, plan.spanD_hi);

    // ---- fuse modes that are contiguous in every tensor that carries them ----
    fuse_modes(plan.batch);
    fuse_modes(plan.m);
    fuse_modes(plan.n);
    fuse_modes(plan.k);

    // ---- roles: D's smallest-stride free mode goes to the M side (commutativity) ----
    {
        int64_t bestM = INT64_MAX, bestN = INT64_MAX;
        for (auto &md : plan.m) bestM = std::min(bestM, iabs(md.sD));
        for (auto &md : plan.n) bestN = std::min(bestN, iabs(md.sD));
        bool swap = bestN < bestM;
        if (plan.m.empty() && !plan.n.empty()) swap = true;
        if (swap) {
            std::swap(plan.m, plan.n);
            for (auto *g : {&plan.batch, &plan.m, &plan.n, &plan.k})
                for (auto &md : *g) std::swap(md.sA, md.sB);
            std::swap(plan.conjA, plan.conjB);
            std::swap(plan.cplxA, plan.cplxB);
            plan.swapped = true;
        }
    }

    // ---- loop order: D decides the order of the free and batch modes ----
    auto by_sD = [](const Mode &x, const Mode &y) { return iabs(x.sD) < iabs(y.sD); };
    std::stable_sort(plan.m.begin(), plan.m.end(), by_sD);
    std::stable_sort(plan.n.begin(), plan.n.end(), by_sD);
    std::stable_sort(plan.batch.begin(), plan.batch.end(), by_sD);

    // When D's fastest free mode x is far apart in the input (rows of a tile would each start in
    // a different DRAM page) and the input has a closer free mode y, block the two: a tile's rows
    // become x_in (one 32-byte sector of D) times y_in (neighbouring rows of the input), so both
    // the input reads and the D writes move whole sectors.  Splitting a mode is only a
    // re-indexing: the outer parts follow as modes of their own.
    const int64_t esz0 = int64_t(dtype_size(plan.dtype));
    auto block_free_modes = [&](std::vector<Mode> &g, bool forA) {
        if (g.size() < 2) return;
        auto S = [&](const Mode &md) { return iabs(forA ? md.sA : md.sB); };
        size_t y = 1;
        for (size_t i = 2; i < g.size(); ++i)
            if (S(g[i]) < S(g[y])) y = i;
        if (S(g[0]) < 1024 || S(g[y]) * 8 > S(g[0])) return;      // x is close enough, or y no better
        const int64_t x_in = largest_divisor_at_most(g[0].extent, std::max<int64_t>(1, 32 / esz0));
        const int64_t y_in = largest_divisor_at_most(g[y].extent, std::max<int64_t>(1, 128 / x_in));
        if (y_in < 2) return;
        Mode xi = g[0], xo = g[0], yi = g[y], yo = g[y];
        xi.extent = x_in; xo.extent = g[0].extent / x_in;
        xo.sA *= x_in; xo.sB *= x_in; xo.sD *= x_in;
        yi.extent = y_in; yo.extent = g[y].extent / y_in;
        yo.sA *= y_in; yo.sB *= y_in; yo.sD *= y_in;
        std::vector<Mode> out = {xi, yi};
        if (xo.extent > 1) out.push_back(xo);
        if (yo.extent > 1) out.push_back(yo);
        for (size_t i = 1; i < g.size(); ++i)
            if (i != y) out.push_back(g[i]);
        g = out;
    };
    block_free_modes(plan.m, true);
    block_free_modes(plan.n, false);
    // The N-side input's stride-1 mode, when it is a free mode that D happens to place late (and no
    // contracted mode is contiguous in that input), comes first among the N modes: the input can then
    // be fetched in 16-byte pieces along it.  The order of the N modes only decides which columns of D
    // share a tile; D itself is written along the M modes.
    {
        bool k_contiguous = false;
        for (auto &md : plan.k) k_contiguous = k_contiguous || iabs(md.sB) == 1;
        if (!k_contiguous)
            for (size_t i = 1; i < plan.n.size(); ++i)
                if (iabs(plan.n[i].sB) == 1 && plan.n[i].extent % 4 == 0) {
                    std::rotate(plan.n.begin(), plan.n.begin() + long(i), plan.n.begin() + long(i) + 1);
                    break;
                }
    }

    // which direction of each input tile is closest to contiguous in memory
    auto min_k_stride = [&](bool forA, int &where) {
        int64_t best = INT64_MAX;
        where = -1;
        for (size_t i = 0; i < plan.k.size(); ++i) {
            const int64_t s = iabs(forA ? plan.k[i].sA : plan.k[i].sB);
            if (s < best) { best = s; where = int(i); }
        }
        return best;
    };
    int kA = -1, kB = -1;
    const int64_t minKA = min_k_stride(true, kA), minKB = min_k_stride(false, kB);
    const int64_t freeA = plan.m.empty() ? INT64_MAX : iabs(plan.m[0].sA);
    const int64_t freeB = plan.n.empty() ? INT64_MAX : iabs(plan.n[0].sB);
    plan.dirA = (freeA <= minKA) ? LoadDir::ALONG_FREE : LoadDir::ALONG_K;
    plan.dirB = (freeB <= minKB) ? LoadDir::ALONG_FREE : LoadDir::ALONG_K;

    // contracted modes: the mode an input wants to run along comes first; when A and B want
    // different ones both are split so that a K tile holds a small box of each
    {
        const bool needA = plan.dirA == LoadDir::ALONG_K, needB = plan.dirB == LoadDir::ALONG_K;
        std::vector<Mode> ordered;
        std::vector<Mode> rest = plan.k;
        auto take = [&](int idx) { ordered.push_back(rest[size_t(idx)]); rest.erase(rest.begin() + idx); };
        if (needA && needB && kA != kB) {
            const int64_t fa = largest_divisor_at_most(rest[size_t(kA)].extent, 4);
            const int64_t fb = largest_divisor_at_most(rest[size_t(kB)].extent, 4);
            if (fa > 1 && fb > 1) {
                split_mode(rest, size_t(kA), fa);
                split_mode(rest, size_t(kB), fb);
            }
            take(kA);
            take(kB > kA ? kB - 1 : kB);
        } else if (needA) {
            take(kA);
        } else if (needB) {
            take(kB);
        }
        const bool sortA = needA || !needB;
        std::stable_sort(rest.begin(), rest.end(), [&](const Mode &x, const Mode &y) {
            return sortA ? iabs(x.sA) < iabs(y.sA) : iabs(x.sB) < iabs(y.sB);
        });
        ordered.insert(ordered.end(), rest.begin(), rest.end());
        plan.k = ordered;
    }

    plan.Bt = product(plan.batch);
    plan.M = product(plan.m);
    plan.N = product(plan.n);
    plan.K = product(plan.k);

    // ---- vector width the strides allow for each input (elements per 16-byte load) ----
    const int64_t esz = int64_t(dtype_size(plan.dtype));
    auto vec_for = [&](bool forA, LoadDir dir) -> int32_t {
        const std::vector<Mode> &fastg = (dir == LoadDir::ALONG_FREE) ? (forA ? plan.m : plan.n) : plan.k;
        if (fastg.empty()) return 1;
        auto S = [&](const Mode &md) { return forA ? md.sA : md.sB; };
        for (int64_t v = 16 / esz; v > 1; v /= 2) {
            bool ok = S(fastg[0]) == 1 && fastg[0].extent % v == 0;
            auto others_ok = [&](const std::vector<Mode> &g, size_t from) {
                for (size_t i = from; i < g.size(); ++i)
                    if (S(g[i]) % v) return false;
                return true;
            };
            const std::vector<Mode> &freeg = forA ? plan.m : plan.n;
            ok = ok && others_ok(freeg, dir == LoadDir::ALONG_FREE ? 1 : 0);
            ok = ok && others_ok(plan.k, dir == LoadDir::ALONG_K ? 1 : 0);
            ok = ok && others_ok(plan.batch, 0);
            if (ok) return int32_t(v);
        }
        return 1;
    };
    plan.vecA = vec_for(true, plan.dirA);
    plan.vecB = vec_for(false, plan.dirB);
    plan.alignA = plan.vecA * esz;
    plan.alignB = plan.vecB * esz;
    // consecutive m that are consecutive in D: lets the fp32 epilogue store 16 bytes at a time
    plan.vecD = 1;
    if (esz == 4 && !plan.m.empty() && plan.m[0].sD == 1 && plan.m[0].extent % 4 == 0) {
        bool ok = true;
        for (size_t i = 1; i < plan.m.size(); ++i) ok = ok && plan.m[i].sD % 4 == 0;
        for (auto &md : plan.n) ok = ok && md.sD % 4 == 0;
        for (auto &md : plan.batch) ok = ok && md.sD % 4 == 0;
        if (ok) plan.vecD = 4;
    }

    {
        const int64_t v = 16 / esz;          // elements in 16 bytes (1 for complex128: always whole)
        auto rows16 = [&](bool inD) {
            auto S = [&](const Mode &md) { return inD ? md.sD : md.sA; };
            if (v == 1) return true;
            if (plan.m.empty() || S(plan.m[0]) != 1 || plan.m[0].extent % v != 0) return false;
            for (size_t i = 1; i < plan.m.size(); ++i) if (S(plan.m[i]) % v) return false;
            for (auto &md : plan.batch) if (S(md) % v) return false;
            for (auto &md : (inD ? plan.n : plan.k)) if (S(md) % v) return false;
            return true;
        };
        plan.rows16D = rows16(true);
        plan.rows16A = rows16(false);
    }

    // ---- kernel choice ----
    const int64_t entries = 2 * (plan.M + plan.N + plan.K) + 3 * plan.Bt;
    // mixed element types and 32-bit storage with sums kept in fp64 run on the per-element kernel
    const bool wide_sums = req.strict_fp32 == 2 && esz0 == (dtype_is_complex(plan.dtype) ? 8 : 4);
    const bool tiled_ok = !plan.has_isolated && entries <= kMaxTableEntries && !plan.mixed && !wide_sums;
    plan.kernel = BTC_KERNEL_GENERIC;
    if (req.force_kernel == BTC_KERNEL_TILED && !tiled_ok) return BTC_ERR_NOT_SUPPORTED;
    // (with at most four contracted indices the streaming kernel serves every size)
    if (req.force_kernel == BTC_KERNEL_TILED ||
        (req.force_kernel == BTC_KERNEL_AUTO && tiled_ok &&
         (double(plan.M) * double(plan.N) * double(plan.K) * double(plan.Bt) >= 32768.0 || plan.K <= 4)))
        plan.kernel = BTC_KERNEL_TILED;

    if (plan.kernel == BTC_KERNEL_TILED) {
        plan.offA_m = build_table(plan.m, [](const Mode &md) { return md.sA; });
        plan.offD_m = build_table(plan.m, [](const Mode &md) { return md.sD; });
        plan.offB_n = build_table(plan.n, [](const Mode &md) { return md.sB; });
        plan.offD_n = build_table(plan.n, [](const Mode &md) { return md.sD; });
        plan.offA_k = build_table(plan.k, [](const Mode &md) { return md.sA; });
        plan.offB_k = build_table(plan.k, [](const Mode &md) { return md.sB; });
        plan.offA_h = build_table(plan.batch, [](const Mode &md) { return md.sA; });
        plan.offB_h = build_table(plan.batch, [](const Mode &md) { return md.sB; });
        plan.offD_h = build_table(plan.batch, [](const Mode &md) { return md.sD; });
    }
    plan.split_k = 1;
    return BTC_SUCCESS;
}

bool make_tma_operand(const Plan &pl, int bm, int bk, TmaOperand &out)
{
    out = TmaOperand();
    if (pl.m.empty() || pl.k.empty() || dtype_size(pl.dtype) != 4) return false;
    struct Part { int64_t extent, stride, box; int cls, idx; };       // cls 0: M, 1: K, 2: batch
    std::vector<Part> parts;
    int64_t rem = bm;
    for (size_t i = 0; i < pl.m.size(); ++i) {
        Part p{pl.m[i].extent, pl.m[i].sA, 1, 0, int(i)};
        if (rem > 1) {
            if (rem % p.extent == 0) { p.box = p.extent; rem /= p.extent; }
            else if (p.extent % rem == 0) { p.box = rem; rem = 1; }
            else if (pl.m.size() == 1 && p.extent > rem) { p.box = rem; rem = 1; }   // ragged last tile: zero-filled by the copy
            else return false;
        }
        parts.push_back(p);
    }
    if (rem != 1) return false;
    for (size_t i = 0; i < pl.k.size(); ++i) {
        Part p{pl.k[i].extent, pl.k[i].sA, 1, 1, int(i)};
        if (i == 0) {
            if (p.extent % bk != 0 && !(pl.k.size() == 1 && p.extent > bk)) return false;
            p.box = bk;
        }
        parts.push_back(p);
    }
    for (size_t i = 0; i < pl.batch.size(); ++i) parts.push_back(Part{pl.batch[i].extent, pl.batch[i].sA, 1, 2, int(i)});
    for (auto &p : parts)
        if (p.stride <= 0) return false;
    const size_t k0 = pl.m.size();
    if (parts[k0].stride == 1) out.k_major = true;
    else if (parts[0].stride != 1 || parts[0].box == 1) return false;

    // dimensions: the contiguous one, the other parts of the box in shared-memory order, the rest
    struct Dim { int64_t extent, stride, box; std::vector<std::pair<size_t, int64_t>> members; };
    std::vector<Dim> dims;
    auto add = [&](size_t i) { dims.push_back(Dim{parts[i].extent, parts[i].stride, parts[i].box, {{i, 1}}}); };
    if (out.k_major) add(k0);
    for (size_t i = 0; i < pl.m.size(); ++i)
        if (parts[i].box > 1) add(i);
    if (!out.k_major) add(k0);
    for (size_t i = 0; i < parts.size(); ++i)
        if (parts[i].box == 1) add(i);
    for (bool changed = true; changed;) {
        changed = false;
        for (size_t x = 0; x < dims.size() && !changed; ++x)
            for (size_t y = 0; y < dims.size() && !changed; ++y) {
                if (x == y || dims[y].box != 1 || dims[y].stride != dims[x].stride * dims[x].extent) continue;
                for (auto &mb : dims[y].members) dims[x].members.push_back({mb.first, mb.second * dims[x].extent});
                dims[x].extent *= dims[y].extent;
                dims.erase(dims.begin() + y);
                changed = true;
            }
    }
    if (dims.size() > 5) return false;
    out.rank = int32_t(dims.size());
    std::vector<std::pair<int, int64_t>> where(parts.size());        // part -> (dimension, multiplier)
    for (size_t d = 0; d < dims.size(); ++d) {
        if (dims[d].extent >= (int64_t(1) << 31) || dims[d].box > 256) return false;
        if (d > 0 && (dims[d].stride % 4 != 0 || dims[d].stride >= (int64_t(1) << 38))) return false;
        out.dim[d] = uint64_t(dims[d].extent);
        out.stride[d] = uint64_t(dims[d].stride);
        out.box[d] = uint32_t(dims[d].box);
        for (auto &mb : dims[d].members) where[mb.first] = {int(d), mb.second};
    }
    // a bulk copy starts on a 16-byte boundary: along dimension 0 the box and every coordinate
    // step (the multipliers of the loop dimensions that share it) are multiples of four elements
    if (out.box[0] % 4 != 0) return false;
    for (auto &mb : dims[0].members)
        if (mb.second != 1 && mb.second % 4 != 0) return false;
    for (size_t d = dims.size(); d < 5; ++d) out.stride[d] = dims.size() > 1 ? out.stride[dims.size() - 1] : 4;   // extent 1: never stepped

    auto coords_of = [&](int cls, const std::vector<Mode> &g, int64_t lin, int32_t *c) {
        for (int d = 0; d < 5; ++d) c[d] = 0;
        for (size_t i = 0; i < g.size(); ++i) {
            const int64_t idx = lin % g[i].extent;
            lin /= g[i].extent;
            const size_t part = (cls == 0 ? 0 : (cls == 1 ? k0 : k0 + pl.k.size())) + i;
            c[where[part].first] += int32_t(idx * where[part].second);
        }
    };
    const int64_t tiles_m = (pl.M + bm - 1) / bm, stages = (pl.K + bk - 1) / bk;
    out.coordM.resize(size_t(tiles_m) * 5);
    out.coordK.resize(size_t(stages) * 5);
    out.coordH.resize(size_t(pl.Bt) * 5);
    for (int64_t t = 0; t < tiles_m; ++t) coords_of(0, pl.m, t * bm, &out.coordM[size_t(t) * 5]);
    for (int64_t t = 0; t < stages; ++t) coords_of(1, pl.k, t * bk, &out.coordK[size_t(t) * 5]);
    for (int64_t t = 0; t < pl.Bt; ++t) coords_of(2, pl.batch, t, &out.coordH[size_t(t) * 5]);
    out.ok = true;
    return true;
}

void split_isolated(const PlanRequest &req, PlanRequest &inner, IsolatedSum &sumA, IsolatedSum &sumB)
{
    inner = req;
    auto contains = [](const std::vector<int64_t> &v, int64_t x) { return std::find(v.begin(), v.end(), x) != v.end(); };
    auto one = [&](const TensorDesc &X, const std::vector<int64_t> &labX, const std::vector<int64_t> &labOther,
                   TensorDesc &Xr, std::vector<int64_t> &labXr, IsolatedSum &sum) {
        struct U { int64_t label, extent, stride; bool iso; };
        std::vector<U> u;                                   // unique labels, strides of repeats added (Note 6)
        for (size_t i = 0; i < labX.size(); ++i) {
            size_t k = 0;
            while (k < u.size() && u[k].label != labX[i]) ++k;
            if (k == u.size()) u.push_back({labX[i], X.extent[i], 0, !contains(labOther, labX[i]) && !contains(req.labelsD, labX[i])});
            u[k].stride += X.stride[i];
        }
        sum = IsolatedSum();
        for (auto &x : u) sum.active = sum.active || (x.iso && x.extent > 1);
        if (!sum.active) return;
        std::stable_sort(u.begin(), u.end(), [](const U &a, const U &b) { return iabs(a.stride) < iabs(b.stride); });
        Xr.extent.clear(); Xr.stride.clear(); labXr.clear();
        int64_t min_keep = INT64_MAX, min_iso = INT64_MAX;
        for (auto &x : u) {
            if (x.iso) {
                if (x.extent == 1) continue;
                sum.iso_ext.push_back(x.extent); sum.iso_str.push_back(x.stride);
                sum.total_iso *= x.extent;
                min_iso = std::min(min_iso, iabs(x.stride));
            } else {
                sum.keep_ext.push_back(x.extent); sum.keep_str.push_back(x.stride);
                Xr.extent.push_back(x.extent); Xr.stride.push_back(sum.total_keep); labXr.push_back(x.label);
                sum.total_keep *= x.extent;
                if (x.extent > 1) min_keep = std::min(min_keep, iabs(x.stride));
            }
        }
        sum.lanes_over_iso = min_iso < min_keep && sum.total_iso >= 32;
        // neighbours whose strides chain act as one loop dimension (fewer divisions per element);
        // X' keeps the same element order either way
        auto chain = [](std::vector<int64_t> &ext, std::vector<int64_t> &str) {
            size_t w = 0;
            for (size_t i = 0; i < ext.size(); ++i) {
                if (w > 0 && str[i] == str[w - 1] * ext[w - 1]) { ext[w - 1] *= ext[i]; continue; }
                ext[w] = ext[i]; str[w] = str[i]; ++w;
            }
            ext.resize(w); str.resize(w);
        };
        chain(sum.keep_ext, sum.keep_str);
        chain(sum.iso_ext, sum.iso_str);
    };
    one(req.A, req.labelsA, req.labelsB, inner.A, inner.labelsA, sumA);
    one(req.B, req.labelsB, req.labelsA, inner.B, inner.labelsB, sumB);
}

int make_elementwise_plan(const ElementwiseRequest &req, ElementwisePlan &plan)
{
    const TensorDesc &A = req.A, &C = req.C;
    if (A.extent.size() != A.stride.size() || A.extent.size() != req.labelsA.size() ||
        C.extent.size() != C.stride.size() || C.extent.size() != req.labelsC.size())
        return BTC_ERR_INVALID_ARGUMENT;
    if (A.dtype != C.dtype || (req.has_b && req.B.dtype != C.dtype)) return BTC_ERR_NOT_SUPPORTED;
    for (size_t i = 0; i < C.extent.size(); ++i)
        for (size_t j = 0; j < i; ++j)
            if (req.labelsC[i] == req.labelsC[j]) return BTC_ERR_NOT_SUPPORTED;   // would write a diagonal of C only
    if (req.has_b) {
        if (req.B.extent.size() != C.extent.size()) return BTC_ERR_C_D_MISMATCH;
        for (size_t i = 0; i < C.extent.size(); ++i)
            if (req.B.extent[i] != C.extent[i]) return BTC_ERR_C_D_MISMATCH;
    }
    if (d_may_alias(C)) return BTC_ERR_D_ALIASING;

    plan = ElementwisePlan();
    plan.dtype = C.dtype;
    plan.has_b = req.has_b;
    plan.conjA = req.conjA && dtype_is_complex(C.dtype);
    plan.conjB = req.conjB && dtype_is_complex(C.dtype);
    struct Row { int64_t label; Mode m; };
    std::vector<Row> keep, sum;
    for (size_t i = 0; i < C.extent.size(); ++i) {
        Mode m;
        m.extent = C.extent[i];
        m.sD = C.stride[i];
        m.sB = req.has_b ? req.B.stride[i] : 0;
        keep.push_back({req.labelsC[i], m});
    }
    for (size_t i = 0; i < A.extent.size(); ++i) {
        std::vector<Row> *where = &sum;
        size_t k = 0;
        for (k = 0; k < keep.size(); ++k)
            if (keep[k].label == req.labelsA[i]) { where = &keep; break; }
        if (where == &sum) {
            for (k = 0; k < sum.size(); ++k)
                if (sum[k].label == req.labelsA[i]) break;
            if (k == sum.size()) {
                Mode m;
                m.extent = A.extent[i];
                sum.push_back({req.labelsA[i], m});
            }
        }
        if ((*where)[k].m.extent != A.extent[i]) return BTC_ERR_EXTENT_MISMATCH;
        (*where)[k].m.sA += A.stride[i];       // repeated labels add their strides (Note 6)
    }
    for (auto &r : keep) if (r.m.extent > 1) plan.keep.push_back(r.m);
    for (auto &r : sum) if (r.m.extent > 1) plan.sum.push_back(r.m);
    fuse_modes(plan.keep);
    fuse_modes(plan.sum);
    std::stable_sort(plan.keep.begin(), plan.keep.end(), [](const Mode &x, const Mode &y) { return iabs(x.sD) < iabs(y.sD); });
    std::stable_sort(plan.sum.begin(), plan.sum.end(), [](const Mode &x, const Mode &y) { return iabs(x.sA) < iabs(y.sA); });
    plan.total_keep = product(plan.keep);
    plan.total_sum = product(plan.sum);
    span_of(req.A, plan.spanA_lo, plan.spanA_hi);
    if (req.has_b) span_of(req.B, plan.spanB_lo, plan.spanB_hi);
    span_of(req.C, plan.spanC_lo, plan.spanC_hi);

    // When A is read far more contiguously along another dimension than along the one C is
    // written along, go through shared-memory tiles: read along A's dimension, write along C's.
    plan.kernel = ElementwiseKernel::DIRECT;
    if (plan.keep.size() >= 2 && plan.keep[0].extent >= 8) {
        int best = -1;
        for (size_t i = 1; i < plan.keep.size(); ++i)
            if (plan.keep[i].sA != 0 && plan.keep[i].extent >= 8 &&
                (best < 0 || iabs(plan.keep[i].sA) < iabs(plan.keep[size_t(best)].sA)))
                best = int(i);
        const int64_t s0 = iabs(plan.keep[0].sA);
        if (best >= 0 && s0 != 0 && iabs(plan.keep[size_t(best)].sA) * 4 <= s0) {
            plan.kernel = ElementwiseKernel::TRANSPOSING;
            plan.tile_mode_a = best;
        }
    }
    return BTC_SUCCESS;
}

std::string Plan::describe() const
{
    std::ostringstream o;
    auto dump = [&](const char *name, const std::vector<Mode> &g) {
        o << name << "[";
        for (auto &md : g) o << "(" << md.extent << ":" << md.sA << "," << md.sB << "," << md.sD << ")";
        o << "] ";
    };
    o << "dtype=" << int(dtype) << " swapped=" << swapped << " Bt=" << Bt << " M=" << M << " N=" << N
      << " K=" << K << " ";
    dump("H", batch); dump("M", m); dump("N", n); dump("K", k);
    o << "kernel=" << kernel << " tile=" << tile.bm << "x" << tile.bn << "x" << tile.bk
      << " splitK=" << split_k << " dirA=" << int(dirA) << " dirB=" << int(dirB) << " vecA=" << vecA
      << " vecB=" << vecB;
    return o.str();
}

}  // namespace btc
