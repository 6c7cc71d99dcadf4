// Host-side planning for the outer synchronisation: module geometry, contributor sets,
// normalised coefficients and the split of one launch into per-CTA element ranges.
// Pure C++ (no CUDA): the same code serves plan-only contexts.
#pragma once

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <vector>

namespace dipaco {

// Flags of one module's pass inside one launch.
enum : int {
    PASS_UPDATE = 1,       // apply the Nesterov step and store theta', m'
    PASS_PARTIAL_IN = 2,   // start the reduction from the stored partial sum
    PASS_PARTIAL_OUT = 4,  // store the running sum instead of updating
    PASS_CAST_IN = 8,      // write-back only: read cast(theta') from the cast scratch, not fp32 theta'
};

struct ModuleGeom {
    int level = 0, index = 0;
    int64_t theta_off = 0;    // elements into theta / momentum
    int64_t path_off = 0;     // elements into a path copy (start of the level)
    int64_t numel = 0;
    int64_t partial_off = -1; // elements into the partial-sum scratch, -1 = none
    int64_t cast_off = 0;     // elements into the cast scratch (every module has a slot)
    std::vector<int> members; // ascending path ids through this module  (S(l,e))
};

struct Grid {
    int L = 0, P = 0;
    std::vector<int> K;
    std::vector<int64_t> N;
    std::vector<int> table;          // [P*L]
    std::vector<float> weights;      // [P] or empty = uniform
    std::vector<float> module_scale; // [modules] factor on the outer gradient, empty = 1
    std::vector<uint8_t> level_sync; // [L] 0 = level takes no part in the exchange, empty = all do
    std::vector<int> level_first;    // module id of (l,0)
    std::vector<ModuleGeom> modules; // level-major
    int64_t module_params = 0, params_per_path = 0;
    int chunk_paths = 0, num_chunks = 1;
    int64_t scratch_elems = 0;
    int64_t cast_elems = 0;                // size of the cast scratch in path elements
    int shard_index = 0, shard_count = 1;  // this context owns one slab of every module
    bool second_moment = false;            // the optimiser keeps a second state array (Adam family)

    int module_id(int l, int e) const { return level_first[l] + e; }
    bool synced(const ModuleGeom &m) const { return level_sync.empty() || level_sync[(size_t)m.level]; }
    float scale_of(size_t id) const { return module_scale.empty() ? 1.0f : module_scale[id]; }
    // Element range of a module that this shard owns: equal slabs cut at multiples of 8192
    // elements (a multiple of every tile size), the last shard takes the remainder.
    void shard_range(const ModuleGeom &m, int64_t &lo, int64_t &hi) const
    {
        slab_bounds(m.numel, shard_index, shard_count, lo, hi);
    }
    // Slab `index` of `count` of a module of `numel` elements.  Every module of a level has the
    // same size, so the bounds are a property of the level.
    static void slab_bounds(int64_t numel, int index, int count, int64_t &lo, int64_t &hi)
    {
        const int64_t grain = 8192;
        auto cut = [&](int i) -> int64_t {
            if (i <= 0) return 0;
            if (i >= count) return numel;
            const int64_t c = (int64_t)((__int128)numel * i / count);
            return c / grain * grain;
        };
        lo = cut(index);
        hi = cut(index + 1);
    }
    int chunk_of(int path) const { return chunk_paths > 0 ? path / chunk_paths : 0; }
};

// Returns false on invalid arguments.
inline bool build_grid(Grid &g, int L, const int32_t *K, const int64_t *N, int P,
                       const int32_t *table, const float *weights, int chunk_paths)
{
    if (L < 1 || P < 1 || !K || !N || !table || chunk_paths < 0) return false;
    g.L = L; g.P = P;
    g.K.assign(K, K + L);
    g.N.assign(N, N + L);
    for (int l = 0; l < L; ++l)
        if (g.K[l] < 1 || g.N[l] < 0) return false;
    g.table.assign(table, table + (size_t)P * L);
    for (int i = 0; i < P; ++i)
        for (int l = 0; l < L; ++l) {
            int e = g.table[(size_t)i * L + l];
            if (e < 0 || e >= g.K[l]) return false;
        }
    g.weights.clear();
    if (weights) {
        for (int i = 0; i < P; ++i)
            if (!(weights[i] >= 0.0f) || !std::isfinite(weights[i])) return false;
        g.weights.assign(weights, weights + P);
    }
    g.chunk_paths = chunk_paths;
    g.num_chunks = chunk_paths > 0 ? (P + chunk_paths - 1) / chunk_paths : 1;

    g.level_first.resize(L);
    g.modules.clear();
    int64_t theta_off = 0, path_off = 0;
    for (int l = 0; l < L; ++l) {
        g.level_first[l] = (int)g.modules.size();
        for (int e = 0; e < g.K[l]; ++e) {
            ModuleGeom m;
            m.level = l; m.index = e;
            m.theta_off = theta_off; m.path_off = path_off; m.numel = g.N[l];
            theta_off += g.N[l];
            g.modules.push_back(m);
        }
        path_off += g.N[l];
    }
    g.module_params = theta_off;
    g.params_per_path = path_off;
    for (int i = 0; i < P; ++i)
        for (int l = 0; l < L; ++l)
            g.modules[g.module_id(l, g.table[(size_t)i * L + l])].members.push_back(i);

    // partial-sum scratch for the modules whose paths span more than one chunk; a slot for every
    // module in the cast scratch (both kept 16-byte aligned for vector / bulk access)
    g.scratch_elems = 0;
    g.cast_elems = 0;
    for (auto &m : g.modules) {
        // A module's slot in either scratch starts where its theta starts within a group of eight
        // elements (at a multiple of eight when theta_off is one): an element range cut so that
        // theta is 32-byte aligned is then 16-byte aligned in the partial sums (fp32) and in the
        // cast scratch (path type) too.
        m.cast_off = g.cast_elems + (m.theta_off & 7);
        g.cast_elems = (m.cast_off + m.numel + 7) / 8 * 8;
        m.partial_off = -1;
        if (g.num_chunks > 1 && !m.members.empty() &&
            g.chunk_of(m.members.front()) != g.chunk_of(m.members.back())) {
            m.partial_off = g.scratch_elems + (m.theta_off & 7);
            g.scratch_elems = (m.partial_off + m.numel + 7) / 8 * 8;
        }
    }
    return true;
}

// Contributor set and normalised coefficients of one module under a mask.
struct ModuleCoeffs {
    std::vector<int> contributors; // ascending path ids in R(l,e)
    std::vector<float> coeff;      // w_i / W rounded to fp32 (normalised in double)
    bool update = false;           // false: nobody reported or W == 0
};

inline void module_coeffs(const Grid &g, const ModuleGeom &m, const uint8_t *reported,
                          ModuleCoeffs &out)
{
    out.contributors.clear();
    out.coeff.clear();
    double W = 0.0;
    for (int i : m.members) {
        if (reported && !reported[i]) continue;
        out.contributors.push_back(i);
        W += g.weights.empty() ? 1.0 : (double)g.weights[i];
    }
    out.update = !out.contributors.empty() && W > 0.0;
    if (!out.update) {
        out.contributors.clear();
        return;
    }
    for (int i : out.contributors) {
        double w = g.weights.empty() ? 1.0 : (double)g.weights[i];
        out.coeff.push_back((float)(w / W));
    }
}

// One module's work inside one launch, before pointers are resolved.
struct PassSpec {
    int module = 0;
    int flags = 0;
    std::vector<int> contributors; // path ids read in this launch
    std::vector<float> coeff;
    std::vector<int> members;      // path ids written in this launch
    int64_t begin = 0, end = -1;   // element range of the module ([0, numel) when end < 0)
    float scale = 1.0f;            // factor on the finished outer gradient (used with PASS_UPDATE)
    bool second_moment = false;    // the update also reads and writes v (Adam family)
    bool cast_out = false;         // cast(theta') is also stored in the module's cast-scratch slot
};

// Resident mode: one launch covers every module completely.
inline void plan_resident(const Grid &g, const std::vector<ModuleCoeffs> &mc,
                          std::vector<PassSpec> &out)
{
    out.clear();
    for (size_t id = 0; id < g.modules.size(); ++id) {
        const ModuleGeom &m = g.modules[id];
        if (m.members.empty() || m.numel == 0 || !g.synced(m)) continue;
        PassSpec p;
        p.module = (int)id;
        g.shard_range(m, p.begin, p.end);
        if (p.begin >= p.end) continue;
        p.scale = g.scale_of(id);
        p.flags = mc[id].update ? PASS_UPDATE : 0;
        p.second_moment = g.second_moment;
        p.contributors = mc[id].contributors;
        p.coeff = mc[id].coeff;
        p.members = m.members;
        out.push_back(std::move(p));
    }
}

// Chunked mode, accumulate launch of chunk c.  The pass that sees a module's last reporting path
// finishes the module and writes cast(theta') into the chunk's copies; with scatter_all (every
// path copy is on the device: the one-call form) into every copy of the module, whatever its
// chunk; with keep_cast also into the module's cast-scratch slot for later write-back launches.
inline void plan_accumulate(const Grid &g, const std::vector<ModuleCoeffs> &mc, int c,
                            std::vector<PassSpec> &out, bool scatter_all = false,
                            bool keep_cast = false)
{
    out.clear();
    for (size_t id = 0; id < g.modules.size(); ++id) {
        const ModuleGeom &m = g.modules[id];
        const ModuleCoeffs &k = mc[id];
        if (!k.update || m.numel == 0 || !g.synced(m)) continue;
        const int first = g.chunk_of(k.contributors.front());
        const int last = g.chunk_of(k.contributors.back());
        PassSpec p;
        p.module = (int)id;
        g.shard_range(m, p.begin, p.end);
        if (p.begin >= p.end) continue;
        p.scale = g.scale_of(id);
        for (size_t j = 0; j < k.contributors.size(); ++j)
            if (g.chunk_of(k.contributors[j]) == c) {
                p.contributors.push_back(k.contributors[j]);
                p.coeff.push_back(k.coeff[j]);
            }
        if (p.contributors.empty()) continue;
        if (c > first) p.flags |= PASS_PARTIAL_IN;
        if (c == last) {
            p.flags |= PASS_UPDATE;
            p.second_moment = g.second_moment;
            p.cast_out = keep_cast;
            for (int i : m.members)
                if (scatter_all || g.chunk_of(i) == c) p.members.push_back(i);
        } else {
            p.flags |= PASS_PARTIAL_OUT;
        }
        out.push_back(std::move(p));
    }
}

// Chunked mode, write-back launch of chunk c: every slot of the chunk, or (skip_final) only
// those that the accumulate launch of the same chunk did not already fill with the final value.
// With use_cast the modules that were updated this round are filled from their cast-scratch slot
// (path dtype) instead of from fp32 theta'.
inline void plan_writeback(const Grid &g, const std::vector<ModuleCoeffs> &mc, int c, bool skip_final,
                           std::vector<PassSpec> &out, bool use_cast = false)
{
    out.clear();
    for (size_t id = 0; id < g.modules.size(); ++id) {
        const ModuleGeom &m = g.modules[id];
        const ModuleCoeffs &k = mc[id];
        if (m.numel == 0 || !g.synced(m)) continue;
        if (skip_final && k.update && g.chunk_of(k.contributors.back()) == c) continue;
        PassSpec p;
        p.module = (int)id;
        g.shard_range(m, p.begin, p.end);
        if (p.begin >= p.end) continue;
        p.flags = (use_cast && k.update) ? PASS_CAST_IN : 0;
        for (int i : m.members)
            if (g.chunk_of(i) == c) p.members.push_back(i);
        if (p.members.empty()) continue;
        out.push_back(std::move(p));
    }
}

// One-call chunked mode: the modules that nobody updates this round (no reporting path, or zero
// total weight) still hand cast(theta) to every one of their paths.
inline void plan_refill_unchanged(const Grid &g, const std::vector<ModuleCoeffs> &mc,
                                  std::vector<PassSpec> &out)
{
    for (size_t id = 0; id < g.modules.size(); ++id) {
        const ModuleGeom &m = g.modules[id];
        if (mc[id].update || m.members.empty() || m.numel == 0 || !g.synced(m)) continue;
        PassSpec p;
        p.module = (int)id;
        g.shard_range(m, p.begin, p.end);
        if (p.begin >= p.end) continue;
        p.flags = 0;
        p.members = m.members;
        out.push_back(std::move(p));
    }
}

// A contiguous element range of one pass, processed by one CTA.
struct Segment {
    int32_t pass;
    int32_t pad;
    int64_t begin, end;
};

// Bytes one element of a pass moves (cost model for balancing CTAs).
inline double pass_cost_per_elem(const PassSpec &p, int elem_size)
{
    double c = (p.flags & PASS_CAST_IN) ? (double)elem_size : 4.0; // cast slot, or theta, read
    c += (double)elem_size * (double)(p.contributors.size() + p.members.size());
    if (p.cast_out) c += (double)elem_size;
    if (p.flags & PASS_UPDATE) c += 12.0;      // momentum read, theta' and m' written
    if ((p.flags & PASS_UPDATE) && p.second_moment) c += 8.0;  // v read and written
    if (p.flags & PASS_PARTIAL_IN) c += 4.0;
    if (p.flags & PASS_PARTIAL_OUT) c += 4.0;
    return c;
}

// Split [0, full_tiles*tile) of every pass in `which` over num_ctas CTAs with equal cost, cutting
// at tile boundaries.  cta_first has num_ctas+1 entries indexing into segs.
// Range i belongs to pass (*pass_of)[i], or to pass i when pass_of is null (one range per pass).
inline void split_segments(const std::vector<PassSpec> &passes, const std::vector<int64_t> &begin,
                           const std::vector<int64_t> &end, int elem_size, int64_t tile,
                           int num_ctas, std::vector<Segment> &segs, std::vector<int32_t> &cta_first,
                           const std::vector<int32_t> *pass_of = nullptr)
{
    segs.clear();
    cta_first.assign((size_t)num_ctas + 1, 0);
    const size_t ranges = begin.size();
    auto pass_index = [&](size_t i) -> size_t { return pass_of ? (size_t)(*pass_of)[i] : i; };
    double total = 0.0;
    for (size_t i = 0; i < ranges; ++i)
        total += pass_cost_per_elem(passes[pass_index(i)], elem_size) * (double)(end[i] - begin[i]);
    if (total <= 0.0 || num_ctas < 1) return;
    // CTA b ends at the tile boundary nearest to the cumulative cost (b+1)*share, so rounding
    // does not pile up on the last CTA.  A CTA may end up empty on very small launches.
    const double share = total / num_ctas;
    int cta = 0;
    double cum = 0.0;  // cost of everything handed out so far
    cta_first[0] = 0;
    for (size_t i = 0; i < ranges; ++i) {
        const double per_tile = pass_cost_per_elem(passes[pass_index(i)], elem_size) * (double)tile;
        int64_t pos = begin[i];
        while (pos < end[i]) {
            const int64_t tiles_left = (end[i] - pos + tile - 1) / tile;
            int64_t take = tiles_left;
            if (cta < num_ctas - 1) {
                const double target = share * (double)(cta + 1);
                take = (int64_t)std::floor((target - cum) / per_tile + 0.5);
                if (take > tiles_left) take = tiles_left;
                if (take < 1) { // this CTA is full: move on
                    ++cta; cta_first[cta] = (int32_t)segs.size();
                    continue;
                }
            }
            const int64_t stop = std::min(end[i], pos + take * tile);
            segs.push_back(Segment{(int32_t)pass_index(i), 0, pos, stop});
            cum += per_tile * (double)take;
            pos = stop;
        }
    }
    for (int b = cta + 1; b <= num_ctas; ++b) cta_first[b] = (int32_t)segs.size();
}

} // namespace dipaco
