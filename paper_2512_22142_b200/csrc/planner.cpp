// Host planner: GEMM -> sub-GEMM tasks under the cost model of Section 4.1, the uniform grid, and
// the churn re-plan of Section 4.2.  Integer arithmetic only (128-bit intermediates).
//
// The paper solves the plan as a MILP with a commercial solver; this is a deterministic heuristic
// for the same objective and constraints:
//   water-fill a makespan T* at which the devices' capacities (largest area each can finish in T*
//   under downlink, uplink, compute and memory) add up to the work; sort the devices that can take
//   at least one granule cell (the others stay idle: zero-task rule); group them into teams of S
//   (one member per K-slice); deal the teams to column strips in snake order; apportion strip
//   widths and team heights in granules by largest remainder; cut every rectangle into its S
//   K-slices; split whatever still violates the memory constraint.
#include <algorithm>
#include <array>
#include <cmath>
#include <cstring>
#include <map>
#include <numeric>

#include "plan_internal.hpp"

namespace cleave {
namespace {

typedef unsigned __int128 u128;
const uint64_t kNs = 1000000000ull;
const uint64_t kTmax = 1ull << 50;

inline uint64_t cdiv(uint64_t a, uint64_t b) { return (a + b - 1) / b; }
// most numerators fit 64 bits: take the hardware division then (the 128-bit one is a library call)
inline u128 cdiv128(u128 a, u128 b) {
    if (!(a >> 63) && !(b >> 63)) return ((uint64_t)a + (uint64_t)b - 1) / (uint64_t)b;
    return (a + b - 1) / b;
}
inline uint64_t sat64(u128 x) { return x > (u128)UINT64_MAX ? UINT64_MAX : (uint64_t)x; }

// ---- cost model (Section 4.1) ---------------------------------------------------------------
uint64_t cost_dl(uint64_t a, uint64_t b, uint64_t k, const cleave_device_t& d, uint32_t bin, bool lat) {
    u128 t = cdiv128((u128)(a + b) * k * bin * kNs, d.dl_Bps);
    return sat64(t + (lat ? d.dl_lat_ns : 0));
}
uint64_t cost_ul(uint64_t a, uint64_t b, const cleave_device_t& d, uint32_t bout) {
    return sat64(cdiv128((u128)a * b * bout * kNs, d.ul_Bps) + d.ul_lat_ns);
}
uint64_t cost_comp(uint64_t a, uint64_t b, uint64_t k, const cleave_device_t& d) {
    return sat64(cdiv128((u128)2 * a * b * k * 1000, d.flops_mflops));
}
uint64_t cost_task(uint64_t a, uint64_t b, uint64_t k, const cleave_device_t& d, const cleave_plan_opts_t& o) {
    return std::max(std::max(cost_dl(a, b, k, d, o.b_in, true), cost_ul(a, b, d, o.b_out)), cost_comp(a, b, k, d));
}
u128 mem_task(uint64_t a, uint64_t b, uint64_t k, const cleave_plan_opts_t& o) {
    return (u128)(a + b) * k * o.b_in + (u128)a * b * o.b_out;
}

// Side of the largest square block that fits the device's memory with slices of depth kh.
uint64_t square_side_in_memory(uint64_t mem, uint64_t kh, const cleave_plan_opts_t& o) {
    uint64_t lo = 0, hi = 1ull << 32;
    while (lo < hi) {
        uint64_t mid = lo + (hi - lo + 1) / 2;
        u128 need = (u128)2 * mid * kh * o.b_in + (u128)mid * mid * o.b_out;
        if (need <= mem) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// Largest output area the device can complete within T for slices of depth kh.
uint64_t capacity_at(const cleave_device_t& d, uint64_t T, uint64_t kh, uint64_t side, const cleave_plan_opts_t& o) {
    u128 best = (u128)side * side;                                     // memory
    u128 a_comp = (u128)T * d.flops_mflops / ((u128)2000 * kh);        // compute
    best = std::min(best, a_comp);
    u128 a_ul = 0;                                                     // uplink
    if (T > d.ul_lat_ns) a_ul = (u128)(T - d.ul_lat_ns) * d.ul_Bps / ((u128)kNs * o.b_out);
    best = std::min(best, a_ul);
    u128 a_dl = 0;                                                     // downlink: alpha+beta affordable, squared off
    if (T > d.dl_lat_ns) {
        u128 s = (u128)(T - d.dl_lat_ns) * d.dl_Bps / ((u128)kNs * kh * o.b_in);
        a_dl = (s / 2) * (s - s / 2);
    }
    best = std::min(best, a_dl);
    if (best < (u128)o.gran_m * o.gran_n) return 0;                    // cannot take one cell: idle
    return (uint64_t)best;                                             // <= side^2 <= 2^64 - 1
}

uint64_t isqrt64(uint64_t x) {
    uint64_t r = 0, bit = 1ull << 62;
    while (bit > x) bit >>= 2;
    while (bit) {
        if (x >= r + bit) { x -= r + bit; r = (r >> 1) + bit; } else r >>= 1;
        bit >>= 2;
    }
    return r;
}

// total units over weights.size() parts, at least one each, the rest by largest remainder.
std::vector<uint32_t> apportion(uint32_t total, const std::vector<u128>& w) {
    size_t n = w.size();
    u128 W = 0;
    for (u128 x : w) W += x;
    uint32_t rest = total - (uint32_t)n;
    std::vector<uint32_t> q(n);
    std::vector<u128> rem(n);
    uint32_t given = 0;
    for (size_t i = 0; i < n; ++i) {
        u128 prod = (u128)rest * w[i];
        q[i] = (uint32_t)(prod / W);
        rem[i] = prod - (u128)q[i] * W;
        given += q[i];
    }
    std::vector<uint32_t> idx(n);
    std::iota(idx.begin(), idx.end(), 0u);
    std::stable_sort(idx.begin(), idx.end(), [&](uint32_t a, uint32_t b) { return rem[a] > rem[b]; });
    for (uint32_t i = 0; i < rest - given; ++i) q[idx[i]] += 1;
    for (auto& x : q) x += 1;
    return q;
}

std::vector<uint32_t> even_parts(uint32_t total, uint32_t parts) {
    std::vector<uint32_t> v(parts, total / parts);
    for (uint32_t i = 0; i < total % parts; ++i) v[i] += 1;
    return v;
}

struct Rect { uint32_t m0, m1, n0, n1, k0, k1, s, dev; };

int repair_memory(const Rect& r, const cleave_device_t& d, const cleave_plan_opts_t& o, std::vector<Rect>& out) {
    if (mem_task(r.m1 - r.m0, r.n1 - r.n0, r.k1 - r.k0, o) <= (u128)d.mem_bytes) { out.push_back(r); return 0; }
    uint32_t rg = (uint32_t)cdiv(r.m1 - r.m0, o.gran_m), cg = (uint32_t)cdiv(r.n1 - r.n0, o.gran_n);
    Rect a = r, b = r;
    if (rg >= cg && rg > 1) {
        a.m1 = b.m0 = r.m0 + ((rg + 1) / 2) * o.gran_m;
    } else if (cg > 1) {
        a.n1 = b.n0 = r.n0 + ((cg + 1) / 2) * o.gran_n;
    } else {
        return CLEAVE_E_INFEASIBLE;
    }
    int rc = repair_memory(a, d, o, out);
    return rc ? rc : repair_memory(b, d, o, out);
}

// level_cells: output cells of all GEMMs of this GEMM's DAG level together (they run in parallel over the
// same devices, so K is split for fan-out only when the whole level has fewer cells than devices)
int plan_one(const cleave_gemm_t& g, const std::vector<cleave_device_t>& devs, const cleave_plan_opts_t& o, uint64_t level_cells,
             uint32_t* S_out, uint64_t* tstar_out, std::vector<Rect>& rects) {
    const uint32_t D = (uint32_t)devs.size();
    const uint32_t Mg = (uint32_t)cdiv(g.M, o.gran_m), Ng = (uint32_t)cdiv(g.N, o.gran_n), Kg = (uint32_t)cdiv(g.K, o.gran_k);
    uint32_t S, s_limit;
    if (o.ksplit) {
        S = s_limit = std::max(1u, std::min(o.ksplit, Kg));
    } else {
        uint64_t depth = o.kslice_max ? cdiv(g.K, o.kslice_max) : 1;
        uint64_t fan = cdiv(D, level_cells);
        s_limit = std::min(o.ksplit_cap, Kg);
        S = (uint32_t)std::max<uint64_t>(1, std::min<uint64_t>(std::max(depth, fan), s_limit));
    }

    std::vector<uint64_t> side(D), cap(D);
    uint64_t kh = 0, tstar = 0;
    for (;;) {
        kh = std::min<uint64_t>(g.K, (uint64_t)o.gran_k * cdiv(Kg, S));
        for (uint32_t k = 0; k < D; ++k) side[k] = square_side_in_memory(devs[k].mem_bytes, kh, o);
        const u128 need = (u128)S * g.M * g.N;
        auto total = [&](uint64_t T) {
            u128 sum = 0;
            for (uint32_t k = 0; k < D; ++k) sum += capacity_at(devs[k], T, kh, side[k], o);
            return sum;
        };
        if (total(kTmax) >= need) {
            uint64_t lo = 0, hi = kTmax;
            while (lo < hi) {
                uint64_t mid = lo + (hi - lo) / 2;
                if (total(mid) >= need) hi = mid; else lo = mid + 1;
            }
            tstar = lo;
            break;
        }
        if (S + 1 > s_limit) return CLEAVE_E_INFEASIBLE;
        ++S;
    }
    for (uint32_t k = 0; k < D; ++k) cap[k] = capacity_at(devs[k], tstar, kh, side[k], o);

    std::vector<uint32_t> active;
    for (uint32_t k = 0; k < D; ++k) if (cap[k]) active.push_back(k);
    std::stable_sort(active.begin(), active.end(), [&](uint32_t a, uint32_t b) { return cap[a] > cap[b]; });
    const uint32_t n_act = (uint32_t)active.size();
    const uint32_t n_teams = (uint32_t)std::max<uint64_t>(1, std::min<uint64_t>(n_act / S, (uint64_t)Mg * Ng));
    std::vector<u128> weight(n_teams, 0);
    auto member = [&](uint32_t team, uint32_t s) { return active[((uint64_t)team * S + s) % n_act]; };
    for (uint32_t j = 0; j < n_teams; ++j)
        for (uint32_t s = 0; s < S; ++s) weight[j] += cap[member(j, s)];

    uint32_t c = (uint32_t)isqrt64((uint64_t)n_teams * Ng / Mg);
    c = std::max(1u, std::min(c, std::min(n_teams, Ng)));
    while (cdiv(n_teams, c) > Mg) ++c;
    std::vector<std::vector<uint32_t>> strips(c);
    for (uint32_t j = 0; j < n_teams; ++j) {
        uint32_t r = j % (2 * c);
        strips[r < c ? r : 2 * c - 1 - r].push_back(j);
    }
    std::vector<u128> strip_w(c, 0);
    for (uint32_t i = 0; i < c; ++i) {
        if (strips[i].empty() || strips[i].size() > Mg) return CLEAVE_E_INFEASIBLE;
        for (uint32_t j : strips[i]) strip_w[i] += weight[j];
    }
    const std::vector<uint32_t> widths = apportion(Ng, strip_w);
    const std::vector<uint32_t> kparts = even_parts(Kg, S);

    uint32_t col_g = 0;
    for (uint32_t i = 0; i < c; ++i) {
        const uint32_t n0 = col_g * o.gran_n, n1 = (uint32_t)std::min<uint64_t>(g.N, (uint64_t)(col_g + widths[i]) * o.gran_n);
        std::vector<u128> tw;
        for (uint32_t j : strips[i]) tw.push_back(weight[j]);
        const std::vector<uint32_t> heights = apportion(Mg, tw);
        uint32_t row_g = 0;
        for (size_t t = 0; t < strips[i].size(); ++t) {
            const uint32_t m0 = row_g * o.gran_m, m1 = (uint32_t)std::min<uint64_t>(g.M, (uint64_t)(row_g + heights[t]) * o.gran_m);
            uint32_t kg = 0;
            for (uint32_t s = 0; s < S; ++s) {
                Rect r;
                r.m0 = m0; r.m1 = m1; r.n0 = n0; r.n1 = n1;
                r.k0 = kg * o.gran_k;
                r.k1 = (uint32_t)std::min<uint64_t>(g.K, (uint64_t)(kg + kparts[s]) * o.gran_k);
                r.s = s; r.dev = member(strips[i][t], s);
                int rc = repair_memory(r, devs[r.dev], o, rects);
                if (rc) return rc;
                kg += kparts[s];
            }
            row_g += heights[t];
        }
        col_g += widths[i];
    }
    *S_out = S;
    *tstar_out = tstar;
    return 0;
}

inline uint64_t round_up32(uint64_t x) { return (x + 31) / 32 * 32; }

void emit_tasks(cleave_plan_s& p, uint32_t gi, const std::vector<Rect>& rects) {
    std::map<uint32_t, u128> load;
    for (const Rect& r : rects) {
        cleave_task_t t;
        std::memset(&t, 0, sizeof t);
        t.id = t.parent = (uint32_t)p.tasks.size();
        t.gemm = gi; t.dev = r.dev;
        t.m0 = r.m0; t.m1 = r.m1; t.n0 = r.n0; t.n1 = r.n1; t.k0 = r.k0; t.k1 = r.k1;
        t.kslice = r.s; t.flags = 0;
        t.part_off = p.arena_elems;
        t.cost_ns = cost_task(r.m1 - r.m0, r.n1 - r.n0, r.k1 - r.k0, p.devices[r.dev], p.opts);
        p.arena_elems += round_up32((uint64_t)(r.m1 - r.m0) * (r.n1 - r.n0));
        load[r.dev] += t.cost_ns;
        p.tasks.push_back(t);
    }
    u128 worst = 0;
    for (auto& kv : load) worst = std::max(worst, kv.second);
    p.makespan.push_back(sat64(worst));
    p.dead.emplace_back();
}

int validate_common(const cleave_plan_s& p) {
    const cleave_plan_opts_t& o = p.opts;
    if (!o.gran_m || !o.gran_n || !o.gran_k || !o.b_in || !o.b_out || !o.reissue_fanout || !o.ksplit_cap) return CLEAVE_E_INVAL;
    if (o.b_in > 16 || o.b_out > 16) return CLEAVE_E_INVAL;
    if (p.gemms.empty()) return CLEAVE_E_INVAL;
    for (const auto& g : p.gemms) {
        if (!g.M || !g.N || !g.K || g.M >= (1u << 31) || g.N >= (1u << 31) || g.K >= (1u << 31)) return CLEAVE_E_INVAL;
        if (g.transA > 1 || g.transB > 1 || g.level >= 4096) return CLEAVE_E_INVAL;
    }
    return 0;
}

void finish(cleave_plan_s& p) {
    p.n_original = (uint32_t)p.tasks.size();
    p.dropped.assign(p.tasks.size(), 0);
    p.task_ntiles.clear();
    p.tiles.clear();
    build_tiles(p, 0);
    p.tiles_original = (uint32_t)p.tiles.size();
}

}  // namespace

int plan_build(cleave_plan_s& p) {
    int rc = validate_common(p);
    if (rc) return rc;
    if (p.devices.empty()) return CLEAVE_E_NO_DEVICES;
    if (p.opts.tail_alpha_milli) {
        // tail-aware cost (Appendix C): every latency overhead enters with its conditional value-at-risk
        // L * alpha / ((alpha - 1) * beta^(1/alpha)); the factor is fixed to 20 fractional bits, the rest is integer
        if (p.opts.tail_alpha_milli <= 1000 || !p.opts.tail_beta_ppm || p.opts.tail_beta_ppm > 1000000) return CLEAVE_E_INVAL;
        const double a = p.opts.tail_alpha_milli / 1000.0, b = p.opts.tail_beta_ppm / 1000000.0;
        const double f = (a / (a - 1.0)) * std::pow(b, -1.0 / a);
        const uint64_t q = (uint64_t)std::floor(f * 1048576.0);
        for (auto& d : p.devices) {
            if (d.dl_lat_ns > (1ull << 40) || d.ul_lat_ns > (1ull << 40)) return CLEAVE_E_INVAL;
            d.dl_lat_ns = (uint64_t)(((u128)d.dl_lat_ns * q + (1u << 20) - 1) >> 20);
            d.ul_lat_ns = (uint64_t)(((u128)d.ul_lat_ns * q + (1u << 20) - 1) >> 20);
        }
    }
    for (const auto& d : p.devices) {
        if (d.mem_bytes > (1ull << 48) || !d.flops_mflops || d.flops_mflops > (1ull << 40) || !d.dl_Bps ||
            d.dl_Bps > (1ull << 40) || !d.ul_Bps || d.ul_Bps > (1ull << 40) || d.dl_lat_ns > (1ull << 40) ||
            d.ul_lat_ns > (1ull << 40))
            return CLEAVE_E_INVAL;
    }
    std::map<uint32_t, uint64_t> level_cells;
    for (const auto& g : p.gemms) level_cells[g.level] += cdiv(g.M, p.opts.gran_m) * cdiv(g.N, p.opts.gran_n);
    for (uint32_t gi = 0; gi < p.gemms.size(); ++gi) {
        std::vector<Rect> rects;
        uint32_t S = 0; uint64_t tstar = 0;
        rc = plan_one(p.gemms[gi], p.devices, p.opts, level_cells[p.gemms[gi].level], &S, &tstar, rects);
        if (rc) return rc;
        p.ksplit.push_back(S);
        p.tstar.push_back(tstar);
        emit_tasks(p, gi, rects);
    }
    finish(p);
    return build_assembly(p);
}

int plan_build_uniform(cleave_plan_s& p, uint32_t gm, uint32_t gn, uint32_t ks) {
    int rc = validate_common(p);
    if (rc) return rc;
    if (!gm || !gn || !ks) return CLEAVE_E_INVAL;
    for (const auto& g : p.gemms) if (gm > g.M || gn > g.N || ks > g.K) return CLEAVE_E_INVAL;
    if ((u128)gm * gn * ks > (1u << 24)) return CLEAVE_E_INVAL;
    cleave_device_t unit = {1ull << 48, 1000000ull, 1000000000ull, 1000000000ull, 0, 0};
    p.devices.assign((size_t)gm * gn * ks, unit);
    for (uint32_t gi = 0; gi < p.gemms.size(); ++gi) {
        const cleave_gemm_t& g = p.gemms[gi];
        const auto hm = even_parts(g.M, gm), wn = even_parts(g.N, gn), dk = even_parts(g.K, ks);
        std::vector<Rect> rects;
        uint32_t m0 = 0;
        for (uint32_t i = 0; i < gm; ++i) {
            uint32_t n0 = 0;
            for (uint32_t j = 0; j < gn; ++j) {
                uint32_t k0 = 0;
                for (uint32_t s = 0; s < ks; ++s) {
                    Rect r = {m0, m0 + hm[i], n0, n0 + wn[j], k0, k0 + dk[s], s, (uint32_t)rects.size()};
                    rects.push_back(r);
                    k0 += dk[s];
                }
                n0 += wn[j];
            }
            m0 += hm[i];
        }
        p.ksplit.push_back(ks);
        p.tstar.push_back(0);
        emit_tasks(p, gi, rects);
    }
    finish(p);
    return build_assembly(p);
}

// ---- churn recovery (Section 4.2) -------------------------------------------------------------
namespace {
// integers of [lo, hi) outside the union of the intervals
uint32_t uncovered(uint32_t lo, uint32_t hi, std::vector<std::pair<uint32_t, uint32_t>> iv) {
    std::sort(iv.begin(), iv.end());
    uint32_t cur = lo, cov = 0;
    for (auto& x : iv) {
        uint32_t a = std::max(x.first, cur), b = std::min(x.second, hi);
        if (b > a) { cov += b - a; cur = b; }
    }
    return (hi - lo) - cov;
}
}  // namespace

int plan_reissue(cleave_plan_s& p, const uint32_t* failed, uint32_t n, uint32_t* first_new) {
    const cleave_plan_opts_t& o = p.opts;
    *first_new = (uint32_t)p.tasks.size();
    std::vector<uint32_t> F(failed, failed + n);
    std::sort(F.begin(), F.end());
    F.erase(std::unique(F.begin(), F.end()), F.end());
    for (uint32_t f : F) {
        if (f >= p.tasks.size()) return CLEAVE_E_RANGE;
        if (p.tasks[f].flags & CLEAVE_TASK_SUPERSEDED) return CLEAVE_E_INVAL;
    }
    if (F.empty()) return 0;
    std::vector<uint8_t> is_failed(p.tasks.size(), 0);
    for (uint32_t f : F) is_failed[f] = 1;

    struct Span { uint32_t m0, m1, n0, n1, k0, k1; };
    struct Round { std::vector<uint32_t> live; std::set<uint32_t> dead; std::vector<u128> load;   // load, held, first: per live[i]
                   std::map<uint32_t, std::vector<uint32_t>> held_by_dev; std::vector<std::vector<uint32_t>> held;
                   std::vector<Span> first; };                   // ranges of held[i][0]: most survivors hold one task
    std::map<uint32_t, Round> rounds;                     // per affected GEMM
    for (uint32_t f : F) {
        Round& r = rounds[p.tasks[f].gemm];
        r.dead.insert(p.tasks[f].dev);
    }
    for (auto& kv : rounds) {
        Round& r = kv.second;
        r.dead.insert(p.dead[kv.first].begin(), p.dead[kv.first].end());
    }
    for (const cleave_task_t& t : p.tasks) {
        auto it = rounds.find(t.gemm);
        if (it == rounds.end() || (t.flags & CLEAVE_TASK_SUPERSEDED) || is_failed[t.id]) continue;
        if (it->second.dead.count(t.dev)) continue;
        it->second.held_by_dev[t.dev].push_back(t.id);
    }
    for (auto& kv : rounds) {
        for (auto& h : kv.second.held_by_dev) {          // ascending device id
            kv.second.live.push_back(h.first); kv.second.load.push_back(0); kv.second.held.push_back(std::move(h.second));
            const cleave_task_t& t0 = p.tasks[kv.second.held.back()[0]];
            kv.second.first.push_back(Span{t0.m0, t0.m1, t0.n0, t0.n1, t0.k0, t0.k1});
        }
        if (kv.second.live.empty()) return CLEAVE_E_NO_DEVICES;
    }

    std::vector<cleave_task_t> pieces;
    uint32_t next_id = (uint32_t)p.tasks.size();
    for (uint32_t f : F) {
        const cleave_task_t t = p.tasks[f];
        const uint32_t beta = t.n1 - t.n0;
        const uint32_t rows_g = (uint32_t)cdiv(t.m1 - t.m0, o.gran_m);
        const uint32_t parts = std::min(o.reissue_fanout, rows_g);
        uint32_t r0 = t.m0;
        for (uint32_t hg : even_parts(rows_g, parts)) {
            cleave_task_t c = t;
            c.id = next_id++;
            c.parent = f;
            c.dev = UINT32_MAX;
            c.m0 = r0;
            c.m1 = (uint32_t)std::min<uint64_t>(t.m1, (uint64_t)r0 + (uint64_t)hg * o.gran_m);
            c.flags = CLEAVE_TASK_REISSUED;
            c.part_off = t.part_off + (uint64_t)(r0 - t.m0) * beta;
            c.cost_ns = 0;
            pieces.push_back(c);
            r0 = c.m1;
        }
    }

    std::vector<uint32_t> order(pieces.size());
    std::iota(order.begin(), order.end(), 0u);
    auto work = [&](const cleave_task_t& t) { return (u128)2 * (t.m1 - t.m0) * (t.n1 - t.n0) * (t.k1 - t.k0); };
    std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return work(pieces[a]) > work(pieces[b]); });

    auto task_at = [&](uint32_t id) -> const cleave_task_t& {
        return id < p.tasks.size() ? p.tasks[id] : pieces[id - p.tasks.size()];
    };
    // Per GEMM and piece shape the costs that do not depend on what a survivor caches are the same for
    // every piece of that shape: max(uplink, compute), and the full cost when nothing is cached
    // (UINT64_MAX marks a survivor whose memory cannot hold the piece).
    struct ShapeCost { std::vector<uint64_t> ul_comp, full; };
    std::map<std::array<uint32_t, 4>, ShapeCost> shape_costs;
    for (uint32_t pi : order) {
        cleave_task_t& pc = pieces[pi];
        Round& r = rounds[pc.gemm];
        const uint32_t a = pc.m1 - pc.m0, b = pc.n1 - pc.n0, kk = pc.k1 - pc.k0;
        ShapeCost& sc = shape_costs[{pc.gemm, a, b, kk}];
        if (sc.full.empty()) {
            sc.ul_comp.resize(r.live.size());
            sc.full.resize(r.live.size());
            for (size_t li = 0; li < r.live.size(); ++li) {
                const cleave_device_t& d = p.devices[r.live[li]];
                sc.ul_comp[li] = std::max(cost_ul(a, b, d, o.b_out), cost_comp(a, b, kk, d));
                sc.full[li] = mem_task(a, b, kk, o) > (u128)d.mem_bytes ? UINT64_MAX
                                                                         : std::max(cost_dl(a, b, kk, d, o.b_in, false), sc.ul_comp[li]);
            }
        }
        bool found = false;
        u128 best_cand = 0; uint64_t best_cost = 0; size_t best_i = 0;
        for (size_t li = 0; li < r.live.size(); ++li) {
            if (sc.full[li] == UINT64_MAX) continue;
            // rows / columns of the piece this survivor does not hold yet (its own tasks of this GEMM whose
            // K-range contains the piece's); the common case of at most one such task needs no interval union
            const std::vector<uint32_t>& held = r.held[li];
            uint32_t a_hat = a, b_hat = b, n_rel = 0;
            if (held.size() == 1) {                          // the usual case, served from the inline copy
                const Span& h = r.first[li];
                if (h.k0 <= pc.k0 && h.k1 >= pc.k1) {
                    const uint32_t ra = std::max(h.m0, pc.m0), rb = std::min(h.m1, pc.m1);
                    const uint32_t ca = std::max(h.n0, pc.n0), cb = std::min(h.n1, pc.n1);
                    a_hat = a - (rb > ra ? rb - ra : 0u);
                    b_hat = b - (cb > ca ? cb - ca : 0u);
                }
            } else {
                for (uint32_t hid : held) {
                    const cleave_task_t& h = task_at(hid);
                    if (h.k0 <= pc.k0 && h.k1 >= pc.k1) ++n_rel;
                }
            }
            if (n_rel >= 1) {
                std::vector<std::pair<uint32_t, uint32_t>> rows, cols;
                for (uint32_t hid : held) {
                    const cleave_task_t& h = task_at(hid);
                    if (h.k0 <= pc.k0 && h.k1 >= pc.k1) { rows.emplace_back(h.m0, h.m1); cols.emplace_back(h.n0, h.n1); }
                }
                a_hat = uncovered(pc.m0, pc.m1, rows);
                b_hat = uncovered(pc.n0, pc.n1, cols);
            }
            const uint64_t c = (a_hat == a && b_hat == b)
                                   ? sc.full[li]
                                   : std::max(cost_dl(a_hat, b_hat, kk, p.devices[r.live[li]], o.b_in, false), sc.ul_comp[li]);
            const u128 cand = r.load[li] + c;
            if (!found || cand < best_cand) { found = true; best_cand = cand; best_cost = c; best_i = li; }
        }
        if (!found) return CLEAVE_E_INFEASIBLE;
        pc.dev = r.live[best_i];
        pc.cost_ns = best_cost;
        r.load[best_i] += best_cost;
        r.held[best_i].push_back(pc.id);
    }

    for (uint32_t f : F) p.tasks[f].flags |= CLEAVE_TASK_SUPERSEDED;
    for (auto& kv : rounds) p.dead[kv.first] = kv.second.dead;
    p.tasks.insert(p.tasks.end(), pieces.begin(), pieces.end());
    p.dropped.resize(p.tasks.size(), 0);
    build_tiles(p, *first_new);
    return 0;
}

// ---- exec work list -----------------------------------------------------------------------------
// The exec kernel's unit is a pair of half-tiles (128 rows x <= 256 columns each, same GEMM, K-range
// and columns; one CTA of a cluster per half).  Two ways to cut a GEMM into pairs:
//
//   grid      All block edges of the GEMM's tasks lie on multiples of 128 (the default granules): the
//             GEMM is cut, K-range by K-range, on a global grid of 256 x 256 pairs, whatever the
//             blocks' shapes.  Each 128 x 128 quadrant of a pair is the cell of whichever task owns it
//             there and is stored into that task's block, so narrow, short or odd-sized blocks cost
//             no tensor-core work: every pair is full except at the GEMM's edges.
//   per task  Otherwise (and for replacement tasks) every task is cut into half-tiles of its own,
//             <= 256 columns wide, and half-tiles with equal GEMM, K-range and columns share a pair.
//
// Order of the pairs (tiles running at the same time share operand panels in L2): by DAG level,
// GEMM (deepest K-range first), K-range, band of 4096 rows, column, row.  (Walking a GEMM cell by cell, all K-slices of a
// cell in a row, would let the in-kernel sum find the other slices' blocks in L2, but the operand
// panels of all slices then compete for L2: measured 5 % slower on the Llama-7B-shaped layer.)
namespace {

struct HalfKey {
    uint32_t gemm, k0, k1, n_col, cols;
    bool operator==(const HalfKey& o) const { return gemm == o.gemm && k0 == o.k0 && k1 == o.k1 && n_col == o.n_col && cols == o.cols; }
};
struct Half {
    HalfKey key;
    TileHalf h;
    uint32_t kslice;
};

TileSeg no_seg(uint32_t task) {
    TileSeg s;
    s.task = task; s.ld = 0; s.out_off = 0; s.fin = kNoFin; s.live = 0;
    return s;
}

TileDesc tile_header(const cleave_plan_s& p, uint32_t gi, uint32_t k0, uint32_t k1, uint32_t kslice, uint32_t n_col, uint32_t cols,
                     uint32_t split) {
    const cleave_gemm_t& g = p.gemms[gi];
    TileDesc d;
    std::memset(&d, 0, sizeof d);
    d.gemm = gi;
    d.flags = (g.transA ? TILE_A_MN : 0u) | (g.transB ? 0u : TILE_B_MN) | (p.ksplit[gi] == 1 ? TILE_SINGLE : 0u) |
              ((!g.transA || g.M % 64 == 0) ? TILE_A_BIG : 0u) | ((g.transB || g.N % 64 == 0) ? TILE_B_BIG : 0u);
    d.n_col = n_col;
    d.n_mma = ((cols + 15) / 16 * 16) | (cols << 16);
    d.k0 = k0; d.k1 = k1;
    d.ldc = g.N;
    d.level = (uint32_t)g.level | (std::min(p.ksplit[gi], 255u) << 16) | (std::min(kslice, 255u) << 24);
    d.split = split;
    return d;
}

// Grid tiling of GEMM gi over its original tasks `ids`.  Returns false (nothing appended) when the
// GEMM does not qualify.
bool grid_tiles(cleave_plan_s& p, uint32_t gi, const std::vector<uint32_t>& ids) {
    const cleave_gemm_t& g = p.gemms[gi];
    const uint32_t S = p.ksplit[gi];
    const uint32_t Mc = (uint32_t)cdiv(g.M, 128), Nc = (uint32_t)cdiv(g.N, 128);
    if ((uint64_t)Mc * Nc * S > (1ull << 26)) return false;
    std::vector<uint32_t> owner((size_t)Mc * Nc * S, UINT32_MAX);
    std::vector<uint32_t> sk0(S, UINT32_MAX), sk1(S, 0);
    for (uint32_t id : ids) {
        const cleave_task_t& t = p.tasks[id];
        if (t.m0 % 128 || t.n0 % 128 || (t.m1 % 128 && t.m1 != g.M) || (t.n1 % 128 && t.n1 != g.N) || t.kslice >= S) return false;
        if (sk0[t.kslice] == UINT32_MAX) { sk0[t.kslice] = t.k0; sk1[t.kslice] = t.k1; }
        else if (sk0[t.kslice] != t.k0 || sk1[t.kslice] != t.k1) return false;      // one K-range per slice
        for (uint32_t r = t.m0 / 128; r < cdiv(t.m1, 128); ++r)
            for (uint32_t c = t.n0 / 128; c < cdiv(t.n1, 128); ++c) {
                uint32_t& o = owner[((size_t)t.kslice * Mc + r) * Nc + c];
                if (o != UINT32_MAX) return false;
                o = id;
            }
    }
    for (uint32_t o : owner) if (o == UINT32_MAX) return false;
    // cells of the in-kernel K-slice sum: one per 128 x 128 quadrant, the same in every slice
    const bool fin = S >= 2 && S <= 8 && g.N % 4 == 0;
    uint32_t cell0 = 0;
    if (fin) {
        p.gemm_finishable[gi] = 1;
        cell0 = (uint32_t)p.fin_ref0.size();
        for (uint32_t r = 0; r < Mc; ++r)
            for (uint32_t c = 0; c < Nc; ++c) {
                p.fin_ref0.push_back((uint32_t)p.fin_refs.size());
                for (uint32_t s = 0; s < S; ++s) {
                    const cleave_task_t& t = p.tasks[owner[((size_t)s * Mc + r) * Nc + c]];
                    const uint32_t ld = t.n1 - t.n0;
                    p.fin_refs.push_back(FinRef{t.part_off + (uint64_t)(r * 128 - t.m0) * ld + (c * 128 - t.n0), ld, t.id});
                }
            }
    }
    for (uint32_t s = 0; s < S; ++s)
        for (uint32_t tj = 0; tj < cdiv(Nc, 2); ++tj)
            for (uint32_t ti = 0; ti < cdiv(Mc, 2); ++ti) {
                const uint32_t n_col = tj * 256, cols = std::min(256u, g.N - n_col);
                const uint32_t nseg = cols > 128 ? 2u : 1u;
                TileDesc d = tile_header(p, gi, sk0[s], sk1[s], s, n_col, cols, nseg == 2 ? 128u : cols);
                for (uint32_t r = 0; r < 2; ++r) {
                    const uint32_t cr = 2 * ti + r;
                    TileHalf& h = d.h[r];
                    h.m_row = cr * 128;
                    h.rows = cr < Mc ? std::min(128u, g.M - cr * 128) : 0u;
                    for (uint32_t q = 0; q < 2; ++q) {
                        const uint32_t cc = 2 * tj + q;
                        if (!h.rows || q >= nseg) { h.seg[q] = no_seg(0); continue; }
                        const cleave_task_t& t = p.tasks[owner[((size_t)s * Mc + cr) * Nc + cc]];
                        TileSeg& sg = h.seg[q];
                        sg.task = t.id;
                        sg.ld = t.n1 - t.n0;
                        sg.out_off = t.part_off + (uint64_t)(h.m_row - t.m0) * sg.ld + (cc * 128 - t.n0);
                        sg.fin = fin ? cell0 + cr * Nc + cc : kNoFin;
                        sg.live = 0;
                        p.task_ntiles[t.id] += 1;
                    }
                }
                p.tiles.push_back(d);
            }
    return true;
}

// widths of the column tiles of a block of beta columns
void column_tiles(uint32_t beta, std::vector<uint32_t>& w) {
    w.clear();
    const uint32_t nt = (uint32_t)cdiv(beta, 256);
    // full-width tiles first, the remainder last: fewest operand bytes per FLOP
    for (uint32_t j = 0; j < nt; ++j) w.push_back(std::min(256u, beta - j * 256));
}

// Per-task tiling of the listed tasks (all of one GEMM when `cells`: then the GEMM's cells of the
// in-kernel K-slice sum are made here).
void task_tiles(cleave_plan_s& p, const std::vector<uint32_t>& ids, bool cells) {
    std::vector<Half> halves;
    std::vector<uint32_t> widths;
    for (uint32_t id : ids) {
        const cleave_task_t& t = p.tasks[id];
        const uint32_t alpha = t.m1 - t.m0, beta = t.n1 - t.n0;
        column_tiles(beta, widths);
        const uint32_t mh = (uint32_t)cdiv(alpha, 128);
        p.task_ntiles[id] = mh * (uint32_t)widths.size();
        for (uint32_t hi = 0; hi < mh; ++hi) {
            uint32_t col = 0;
            for (uint32_t wj : widths) {
                Half x;
                x.key = HalfKey{t.gemm, t.k0, t.k1, t.n0 + col, wj};
                x.h.m_row = t.m0 + hi * 128;
                x.h.rows = std::min(128u, alpha - hi * 128);
                x.h.seg[0].task = id;
                x.h.seg[0].ld = beta;
                x.h.seg[0].out_off = t.part_off + (uint64_t)hi * 128 * beta + col;
                x.h.seg[0].fin = kNoFin;
                x.h.seg[0].live = 0;
                x.h.seg[1] = no_seg(id);
                x.kslice = t.kslice;
                halves.push_back(x);
                col += wj;
            }
        }
    }
    // cells: the GEMM qualifies when every half-tile position holds exactly one half-tile per K-slice, all of
    // equal shape, and float4 accesses are aligned
    if (cells && !halves.empty()) {
        const uint32_t gi = halves[0].key.gemm, S = p.ksplit[gi];
        if (S >= 2 && S <= 8 && p.gemms[gi].N % 4 == 0) {
            std::vector<uint32_t> idx(halves.size());
            for (uint32_t i = 0; i < idx.size(); ++i) idx[i] = i;
            std::sort(idx.begin(), idx.end(), [&](uint32_t a, uint32_t b) {
                const Half &x = halves[a], &y = halves[b];
                if (x.h.m_row != y.h.m_row) return x.h.m_row < y.h.m_row;
                if (x.key.n_col != y.key.n_col) return x.key.n_col < y.key.n_col;
                return x.kslice < y.kslice;
            });
            bool ok = idx.size() % S == 0;
            for (size_t c = 0; ok && c < idx.size(); c += S)
                for (uint32_t s = 0; ok && s < S; ++s) {
                    const Half &x = halves[idx[c + s]], &x0 = halves[idx[c]];
                    ok = x.kslice == s && x.h.m_row == x0.h.m_row && x.h.rows == x0.h.rows && x.key.n_col == x0.key.n_col &&
                         x.key.cols == x0.key.cols && x.key.n_col % 4 == 0 && x.key.cols % 4 == 0 && x.h.seg[0].ld % 4 == 0 &&
                         x.h.seg[0].out_off % 4 == 0;
                }
            if (ok) {
                p.gemm_finishable[gi] = 1;
                for (size_t c = 0; c < idx.size(); c += S) {
                    const uint32_t cell = (uint32_t)p.fin_ref0.size();
                    p.fin_ref0.push_back((uint32_t)p.fin_refs.size());
                    for (uint32_t s = 0; s < S; ++s) {
                        Half& x = halves[idx[c + s]];
                        x.h.seg[0].fin = cell;
                        p.fin_refs.push_back(FinRef{x.h.seg[0].out_off, x.h.seg[0].ld, x.h.seg[0].task});
                    }
                }
            }
        }
    }
    // pairs: consecutive half-tiles (by row) of the same GEMM, K-range and columns
    std::stable_sort(halves.begin(), halves.end(), [](const Half& a, const Half& b) {
        if (a.key.gemm != b.key.gemm) return a.key.gemm < b.key.gemm;
        if (a.key.k0 != b.key.k0) return a.key.k0 < b.key.k0;
        if (a.key.k1 != b.key.k1) return a.key.k1 < b.key.k1;
        if (a.key.n_col != b.key.n_col) return a.key.n_col < b.key.n_col;
        if (a.key.cols != b.key.cols) return a.key.cols < b.key.cols;
        return a.h.m_row < b.h.m_row;
    });
    for (size_t i = 0; i < halves.size();) {
        const Half& x = halves[i];
        TileDesc d = tile_header(p, x.key.gemm, x.key.k0, x.key.k1, x.kslice, x.key.n_col, x.key.cols, x.key.cols);
        d.h[0] = x.h;
        // each CTA of the pair loads, multiplies and stores its own half, so any two half-tiles may share a pair
        if (i + 1 < halves.size() && halves[i + 1].key == x.key) { d.h[1] = halves[i + 1].h; i += 2; }
        else { d.h[1].m_row = 0; d.h[1].rows = 0; d.h[1].seg[0] = d.h[1].seg[1] = no_seg(x.h.seg[0].task); i += 1; }
        p.tiles.push_back(d);
    }
}

}  // namespace

void build_tiles(cleave_plan_s& p, uint32_t first_task) {
    const uint32_t kBandRows = 4096;
    const bool original = (first_task == 0);
    const size_t begin = p.tiles.size();
    p.task_ntiles.resize(p.tasks.size(), 0);
    if (original) {
        p.n_levels = 1;
        for (const auto& g : p.gemms) p.n_levels = std::max<uint32_t>(p.n_levels, (uint32_t)g.level + 1);
        p.gemm_finishable.assign(p.gemms.size(), 0);
        p.fin_ref0.clear(); p.fin_refs.clear();
    }
    std::vector<std::vector<uint32_t>> by_gemm(p.gemms.size());
    for (uint32_t id = first_task; id < p.tasks.size(); ++id) {
        const cleave_task_t& t = p.tasks[id];
        const cleave_gemm_t& g = p.gemms[t.gemm];
        if ((t.k0 % 64) || ((t.k1 % 64) && t.k1 != g.K) || (g.transA && (t.m0 % 8)) || (!g.transB && (t.n0 % 8)) ||
            (g.lda % 8) || (g.ldb % 8))
            p.exec_unsupported = 1;
        by_gemm[t.gemm].push_back(id);
    }
    for (uint32_t gi = 0; gi < p.gemms.size(); ++gi) {
        if (by_gemm[gi].empty()) continue;
        if (original) {
            const size_t tiles0 = p.tiles.size(), ref0 = p.fin_ref0.size(), refs0 = p.fin_refs.size();
            if (grid_tiles(p, gi, by_gemm[gi])) continue;
            // not on the 128-grid: undo whatever the attempt counted, cut task by task
            p.tiles.resize(tiles0); p.fin_ref0.resize(ref0); p.fin_refs.resize(refs0);
            p.gemm_finishable[gi] = 0;
            for (uint32_t id : by_gemm[gi]) p.task_ntiles[id] = 0;
        }
        task_tiles(p, by_gemm[gi], original);
    }
    // Within a DAG level the GEMMs whose pairs run longest (deepest K-range) come first, so that the pairs
    // handed out last, which decide how long some clusters idle at the end, are the short ones.
    std::vector<uint32_t> depth(p.gemms.size(), 0);
    for (size_t i = begin; i < p.tiles.size(); ++i)
        depth[p.tiles[i].gemm] = std::max(depth[p.tiles[i].gemm], p.tiles[i].k1 - p.tiles[i].k0);
    std::stable_sort(p.tiles.begin() + begin, p.tiles.end(), [&](const TileDesc& a, const TileDesc& b) {
        const uint32_t la = a.level & 0xFFFFu, lb = b.level & 0xFFFFu;
        if (la != lb) return la < lb;
        if (depth[a.gemm] != depth[b.gemm]) return depth[a.gemm] > depth[b.gemm];
        if (a.gemm != b.gemm) return a.gemm < b.gemm;
        if (a.k0 != b.k0) return a.k0 < b.k0;
        const uint32_t ba = a.h[0].m_row / kBandRows, bb = b.h[0].m_row / kBandRows;
        if (ba != bb) return ba < bb;
        if (a.n_col != b.n_col) return a.n_col < b.n_col;
        return a.h[0].m_row < b.h[0].m_row;
    });
}

// ---- assembly work list ---------------------------------------------------------------------------
// All row / column boundaries of a GEMM's original tasks cut C into cells; in a cell every K-slice is
// served by exactly one task.  Neighbouring cells served by the same tasks are merged again, then
// the rectangles are cut into items of whole rows of roughly 16K outputs each.
int build_assembly(cleave_plan_s& p) {
    p.asm_items.clear(); p.asm_refs.clear(); p.asm_groups.clear();
    std::vector<uint32_t> first_item, gemm_sp;       // per GEMM: first item, launch class
    std::vector<std::vector<uint32_t>> by_gemm(p.gemms.size());
    for (uint32_t id = 0; id < p.n_original; ++id) by_gemm[p.tasks[id].gemm].push_back(id);
    for (uint32_t gi = 0; gi < p.gemms.size(); ++gi) {
        first_item.push_back((uint32_t)p.asm_items.size());
        const cleave_gemm_t& g = p.gemms[gi];
        const uint32_t S = p.ksplit[gi];
        std::vector<uint32_t> rc, cc;
        for (uint32_t id : by_gemm[gi]) {
            const cleave_task_t& t = p.tasks[id];
            rc.push_back(t.m0); rc.push_back(t.m1); cc.push_back(t.n0); cc.push_back(t.n1);
        }
        std::sort(rc.begin(), rc.end()); rc.erase(std::unique(rc.begin(), rc.end()), rc.end());
        std::sort(cc.begin(), cc.end()); cc.erase(std::unique(cc.begin(), cc.end()), cc.end());
        const size_t nr = rc.size() - 1, nc = cc.size() - 1;
        std::vector<uint32_t> cell(nr * nc * S, UINT32_MAX);
        for (uint32_t id : by_gemm[gi]) {
            const cleave_task_t& t = p.tasks[id];
            if (t.kslice >= S) return CLEAVE_E_INVAL;
            const size_t r0 = std::lower_bound(rc.begin(), rc.end(), t.m0) - rc.begin();
            const size_t r1 = std::lower_bound(rc.begin(), rc.end(), t.m1) - rc.begin();
            const size_t c0 = std::lower_bound(cc.begin(), cc.end(), t.n0) - cc.begin();
            const size_t c1 = std::lower_bound(cc.begin(), cc.end(), t.n1) - cc.begin();
            for (size_t r = r0; r < r1; ++r)
                for (size_t c = c0; c < c1; ++c) cell[(r * nc + c) * S + t.kslice] = id;
        }
        for (uint32_t x : cell) if (x == UINT32_MAX) return CLEAVE_E_INVAL;   // not a tiling
        (void)g;
        // merge: horizontal runs per cell row, then vertical runs of identical (columns, tasks)
        struct Seg { uint32_t i0, i1, j0, j1; std::vector<uint32_t> tasks; };
        std::vector<Seg> open, done;
        for (size_t r = 0; r < nr; ++r) {
            std::vector<Seg> row;
            for (size_t c = 0; c < nc; ++c) {
                std::vector<uint32_t> ts(cell.begin() + (r * nc + c) * S, cell.begin() + (r * nc + c + 1) * S);
                if (!row.empty() && row.back().tasks == ts && row.back().j1 == cc[c]) row.back().j1 = cc[c + 1];
                else row.push_back(Seg{rc[r], rc[r + 1], cc[c], cc[c + 1], ts});
            }
            std::vector<Seg> next_open;
            for (Seg& s : row) {
                bool merged = false;
                for (Seg& o : open)
                    if (o.i1 == s.i0 && o.j0 == s.j0 && o.j1 == s.j1 && o.tasks == s.tasks) { o.i1 = s.i1; next_open.push_back(o); o.i1 = UINT32_MAX; merged = true; break; }
                if (!merged) next_open.push_back(s);
            }
            for (Seg& o : open) if (o.i1 != UINT32_MAX) done.push_back(o);
            open.swap(next_open);
        }
        for (Seg& o : open) done.push_back(o);
        std::sort(done.begin(), done.end(), [](const Seg& a, const Seg& b) { return a.i0 != b.i0 ? a.i0 < b.i0 : a.j0 < b.j0; });

        bool vec = (g.N % 4 == 0);
        for (const Seg& s : done) {
            const uint32_t ncols = s.j1 - s.j0;
            const uint32_t rows_per = std::max(1u, 16384u / ncols);
            if (s.j0 % 4 || ncols % 4) vec = false;
            for (uint32_t i = s.i0; i < s.i1; i += rows_per) {
                AsmItem it;
                it.gemm = gi; it.i0 = i; it.nrows = std::min(rows_per, s.i1 - i);
                it.j0 = s.j0; it.ncols = ncols; it.ref0 = (uint32_t)p.asm_refs.size(); it.nslices = S; it.pad = 0;
                for (uint32_t sl = 0; sl < S; ++sl) {
                    const cleave_task_t& t = p.tasks[s.tasks[sl]];
                    AsmRef r;
                    r.ld = t.n1 - t.n0;
                    r.off = t.part_off + (uint64_t)(i - t.m0) * r.ld + (s.j0 - t.n0);
                    r.task = t.id;
                    if (r.off % 4 || r.ld % 4) vec = false;
                    p.asm_refs.push_back(r);
                }
                p.asm_items.push_back(it);
            }
        }
        uint32_t sp = 1;
        while (sp < S) sp *= 2;
        gemm_sp.push_back(vec ? sp : 0u);
    }
    first_item.push_back((uint32_t)p.asm_items.size());
    // one launch per class: reorder the items so that each class is contiguous (GEMM order inside)
    std::vector<AsmItem> sorted;
    sorted.reserve(p.asm_items.size());
    for (uint32_t single : {1u, 0u})
        for (uint32_t fin : {1u, 0u})
            for (uint32_t cls : {1u, 2u, 4u, 8u, 16u, 32u, 0u}) {
                const uint32_t item0 = (uint32_t)sorted.size();
                for (uint32_t gi = 0; gi < p.gemms.size(); ++gi)
                    if (gemm_sp[gi] == cls && (p.ksplit[gi] == 1 ? 1u : 0u) == single && (uint32_t)p.gemm_finishable[gi] == fin)
                        sorted.insert(sorted.end(), p.asm_items.begin() + first_item[gi], p.asm_items.begin() + first_item[gi + 1]);
                if (sorted.size() > item0) p.asm_groups.push_back({cls, item0, (uint32_t)sorted.size() - item0, single, fin});
            }
    p.asm_items.swap(sorted);
    return 0;
}

}  // namespace cleave
