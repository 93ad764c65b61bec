// Host-side planning of evo_validate (see plan.h).  No CUDA calls in this file.
#include "plan.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <unordered_map>

namespace evo {

namespace {

struct Key {
    const void* ref;
    uint64_t n;
    int dtype;
    bool operator==(const Key& o) const { return ref == o.ref && n == o.n && dtype == o.dtype; }
};
struct KeyHash {
    size_t operator()(const Key& k) const {
        size_t h = std::hash<const void*>()(k.ref);
        h ^= std::hash<uint64_t>()(k.n) + 0x9e3779b97f4a7c15ull + (h << 6) + (h >> 2);
        h ^= std::hash<int>()(k.dtype) + 0x9e3779b97f4a7c15ull + (h << 6) + (h >> 2);
        return h;
    }
};

// Cost of one (set, tile) item: the tiles it moves (the reference and every member).  Other weightings were
// measured on a ragged, mixed-type population and lost: 16-bit tiles lighter or heavier than fp32 ones, a
// fixed cost per set.
inline uint64_t item_weight(const SetRec& S) { return static_cast<uint64_t>(S.k) + 1; }

int plan_fail(std::string* err, int status, const char* fmt, ...) {
    char buf[256];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    if (err) *err = buf;
    return status;
}

}  // namespace

int build_plan(const void* const* cand_ptrs, const void* ref_ptr, const evo_desc* descs, uint64_t n_desc,
               int dtype, float atol, float rtol, bool want_groups, uint64_t n_group, uint32_t max_ctas,
               Plan* plan, std::string* err, uint32_t accepted_types) {
    if (!(atol >= 0.f) || !(rtol >= 0.f) || std::isinf(atol) || std::isinf(rtol))
        return plan_fail(err, EVO_ERR_ARG, "atol and rtol must be finite and >= 0");
    if (want_groups != (n_group != 0)) return plan_fail(err, EVO_ERR_ARG, "group_pass and n_group must be given together");
    if (n_desc >= (1ull << 31) || n_group >= (1ull << 31)) return plan_fail(err, EVO_ERR_ARG, "too many descriptors");
    if (n_desc > 0 && (!cand_ptrs || !descs)) return plan_fail(err, EVO_ERR_ARG, "cand_ptrs and descs must not be NULL");
    if (max_ctas == 0) return plan_fail(err, EVO_ERR_ARG, "max_ctas must be positive");

    // ---- how many members a set may hold ----
    // Up to kMaxK.  An item (set, tile) is the unit of the cut below, so a CTA's share is only even to
    // within one item; when every CTA gets work but only a few items (a mid-sized population of many
    // tensors per reference), smaller sets give more, lighter items at the price of reading the
    // reference once more per extra set (from L2, mostly).  The same holds with more reason when
    // there are fewer items than CTAs.
    uint32_t cap = kMaxK;
    {
        std::unordered_map<Key, uint32_t, KeyHash> members_of;
        for (uint64_t i = 0; i < n_desc; ++i) {
            const evo_desc& d = descs[i];
            const int dt = d.dtype == -1 ? dtype : d.dtype;
            if (d.n == 0 || dt < 0 || dt > 31 || dtype_bytes(dt) == 0) continue;      // judged below
            members_of[Key{d.ref ? d.ref : ref_ptr, d.n, dt}] += 1;
        }
        auto items_with = [&](uint32_t c) {
            unsigned __int128 items = 0;
            for (const auto& kv : members_of)
                items += static_cast<unsigned __int128>((kv.first.n + kTileElems - 1) / kTileElems) * ((kv.second + c - 1) / c);
            return items;
        };
        if (items_with(kMaxK) >= max_ctas) {
            while (cap > 4 && items_with(cap) < static_cast<unsigned __int128>(6) * max_ctas) cap /= 2;
        } else {
            // Fewer items than CTAs (a small population): a CTA's time is its start-up plus one member after the
            // other, so the members are spread over as many CTAs as there are, down to one member per set.
            while (cap > 1 && items_with(cap) < max_ctas) cap /= 2;
        }
    }

    // ---- sets: tensors with the same (reference, n, dtype), at most `cap` each ----
    std::unordered_map<Key, uint32_t, KeyHash> open;       // key -> set still accepting members
    std::vector<SetRec>& sets = plan->sets;
    sets.clear();
    std::vector<uint32_t> set_of(n_desc);
    for (uint64_t i = 0; i < n_desc; ++i) {
        const evo_desc& d = descs[i];
        const int dt = d.dtype == -1 ? dtype : d.dtype;
        const unsigned long long ii = i;
        if (dt < 0 || dt > 31 || !((accepted_types >> dt) & 1u) || dtype_bytes(dt) == 0)
            return plan_fail(err, EVO_ERR_DTYPE, "descriptor %llu has dtype %d", ii, dt);
        const void* ref = d.ref ? d.ref : ref_ptr;
        if (d.n > 0 && (!ref || !cand_ptrs[i])) return plan_fail(err, EVO_ERR_ARG, "descriptor %llu has a NULL tensor", ii);
        if (d.n > (1ull << 60)) return plan_fail(err, EVO_ERR_ARG, "descriptor %llu is too large", ii);
        const size_t eb = dtype_bytes(dt);
        if (d.n > 0 && (reinterpret_cast<uintptr_t>(ref) % eb || reinterpret_cast<uintptr_t>(cand_ptrs[i]) % eb))
            return plan_fail(err, EVO_ERR_ALIGN, "descriptor %llu is not aligned to %zu bytes", ii, eb);
        if (want_groups && d.group >= n_group)
            return plan_fail(err, EVO_ERR_ARG, "descriptor %llu has group %u >= n_group", ii, d.group);
        const Key key{d.n ? ref : nullptr, d.n, dt};
        auto it = open.find(key);
        uint32_t s;
        if (it == open.end() || sets[it->second].k == cap) {
            s = static_cast<uint32_t>(sets.size());
            SetRec S{};
            S.ref = ref; S.n = d.n; S.k = 0; S.dtype = static_cast<uint32_t>(dt);
            S.vec_ok = (reinterpret_cast<uintptr_t>(ref) % 16 == 0) ? 1u : 0u;
            S.cta_first = 1; S.cta_last = 0;
            sets.push_back(S);
            open[key] = s;
        } else {
            s = it->second;
        }
        sets[s].k += 1;
        if (reinterpret_cast<uintptr_t>(cand_ptrs[i]) % 16) sets[s].vec_ok = 0;
        set_of[i] = s;
    }
    const uint32_t n_sets = static_cast<uint32_t>(sets.size());

    // ---- members ordered by set ----
    uint32_t off = 0;
    for (auto& S : sets) { S.member_off = off; off += S.k; S.k = 0; }
    plan->members.assign(n_desc, MemberRec{});
    for (uint64_t i = 0; i < n_desc; ++i) {
        SetRec& S = sets[set_of[i]];
        plan->members[S.member_off + S.k] = MemberRec{cand_ptrs[i], static_cast<uint32_t>(i), set_of[i]};
        S.k += 1;
    }

    // ---- cut the weighted item list into one contiguous range per CTA ----
    // An item (set, tile) moves k + 1 tiles of kTileBytes: its weight.
    std::vector<uint64_t> tiles(n_sets);
    std::vector<unsigned __int128> prefix(n_sets + 1);
    prefix[0] = 0;
    plan->total_tiles = 0;
    for (uint32_t s = 0; s < n_sets; ++s) {
        tiles[s] = (sets[s].n + kTileElems - 1) / kTileElems;
        plan->total_tiles += tiles[s];
        prefix[s + 1] = prefix[s] + static_cast<unsigned __int128>(tiles[s]) * item_weight(sets[s]);
    }
    const unsigned __int128 total_cost = prefix[n_sets];
    const uint32_t n_ctas = static_cast<uint32_t>(std::min<uint64_t>(max_ctas, plan->total_tiles));
    plan->ranges.clear();
    plan->n_parts = 0;
    if (n_ctas > 0) {
        // boundary b: the item containing cumulative weight b * total / n_ctas
        std::vector<std::pair<uint32_t, uint64_t>> cut(n_ctas + 1);
        uint32_t s = 0;
        for (uint32_t b = 0; b <= n_ctas; ++b) {
            const unsigned __int128 pos = total_cost * b / n_ctas;
            while (s < n_sets && prefix[s + 1] <= pos) ++s;
            if (s == n_sets) cut[b] = {n_sets, 0};
            else cut[b] = {s, static_cast<uint64_t>((pos - prefix[s]) / item_weight(sets[s]))};
        }
        for (uint32_t b = 0; b < n_ctas; ++b) {
            CtaRange R{};
            const uint32_t sb = cut[b].first;
            const uint64_t tb = cut[b].second;
            uint32_t se = cut[b + 1].first;
            uint64_t te = cut[b + 1].second;
            if (se == n_sets || te == 0) {
                // make the end (set, exclusive tile) point inside the last set that has tiles
                uint32_t p = se;
                while (p > 0 && tiles[p - 1] == 0) --p;
                if (p == 0) { se = 0; te = 0; } else { se = p - 1; te = tiles[se]; }
            }
            // Two boundaries can fall into the same item (heavy items, few tiles): such a run
            // is empty and gets no CTA, so that every CTA in [cta_first, cta_last] of a set
            // really holds a partial record for it.
            if (sb == n_sets || sb > se || (sb == se && tb >= te)) continue;
            const uint32_t cta = static_cast<uint32_t>(plan->ranges.size());
            R.s_begin = sb; R.s_end = se; R.t_begin = tb; R.t_end = te;
            R.first_member = sets[sb].member_off;
            R.part_base = plan->n_parts;
            plan->n_parts += sets[se].member_off + sets[se].k - sets[sb].member_off;
            for (uint32_t q = sb; q <= se; ++q) {
                const uint64_t q0 = q == sb ? tb : 0, q1 = q == se ? te : tiles[q];
                if (q0 >= q1) continue;
                if (sets[q].cta_first > sets[q].cta_last) sets[q].cta_first = cta;
                sets[q].cta_last = cta;
            }
            plan->ranges.push_back(R);
        }
    }

    // ---- descriptor lists per candidate id, for the verdicts ----
    plan->group_off.clear();
    plan->group_desc.clear();
    if (want_groups) {
        plan->group_off.assign(n_group + 1, 0);
        for (uint64_t i = 0; i < n_desc; ++i) plan->group_off[descs[i].group + 1] += 1;
        for (uint64_t g = 0; g < n_group; ++g) plan->group_off[g + 1] += plan->group_off[g];
        plan->group_desc.resize(n_desc);
        std::vector<uint32_t> fill(plan->group_off.begin(), plan->group_off.end() - 1);
        for (uint64_t i = 0; i < n_desc; ++i) plan->group_desc[fill[descs[i].group]++] = static_cast<uint32_t>(i);
    }
    return EVO_OK;
}

}  // namespace evo

// Host-only view of the plan, for inspection and tests: what evo_validate would schedule on a
// device running `max_ctas` persistent CTAs.  Touches no device and dereferences no tensor.
extern "C" EVO_API int evo_plan_inspect(const void* const* cand_ptrs, const void* ref_ptr, const evo_desc* descs,
                                        uint64_t n_desc, int dtype, uint32_t max_ctas, evo_plan_summary* summary,
                                        evo_plan_range* ranges, uint32_t* set_of_desc, uint32_t* set_k) {
    if (!summary) return EVO_ERR_ARG;
    evo::Plan plan;
    std::string err;
    const int st = evo::build_plan(cand_ptrs, ref_ptr, descs, n_desc, dtype, 0.f, 0.f, false, 0, max_ctas, &plan, &err);
    if (st != EVO_OK) return st;
    summary->n_sets = static_cast<uint32_t>(plan.sets.size());
    summary->n_ctas = static_cast<uint32_t>(plan.ranges.size());
    summary->n_parts = plan.n_parts;
    summary->tile_elems = evo::kTileElems;
    summary->total_tiles = plan.total_tiles;
    if (ranges) {
        for (size_t b = 0; b < plan.ranges.size(); ++b) {
            const evo::CtaRange& R = plan.ranges[b];
            ranges[b].set_begin = R.s_begin; ranges[b].set_end = R.s_end;
            ranges[b].tile_begin = R.t_begin; ranges[b].tile_end = R.t_end;
        }
    }
    if (set_of_desc) for (const evo::MemberRec& m : plan.members) set_of_desc[m.desc] = m.set;
    if (set_k) for (size_t s = 0; s < plan.sets.size(); ++s) set_k[s] = plan.sets[s].k;
    return EVO_OK;
}
