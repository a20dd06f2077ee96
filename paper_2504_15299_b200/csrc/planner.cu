// Host-side planning of the bit-width-aware I/O-compute pipeline (Section 3.4): the Hottest-Expert-Bit-First
// load order, the two-queue pipeline model of Eq. 6, and one layer step of the memory-budget scheduler
// (Algorithm 2).  Plain host code: no kernel, no device memory, no allocation visible to the caller.
#include "../../include/d2moe.h"

#include <algorithm>
#include <vector>

namespace {

// requests that read segment k of expert j: every request at width index >= k
inline long long reuse_count(const int32_t* B, int K, int j, int k) {
    long long n = 0;
    for (int kk = k; kk < K; ++kk) n += B[j * K + kk];
    return n;
}

inline int last_requested(const int32_t* B, int K, int j) {
    int last = -1;
    for (int k = 0; k < K; ++k)
        if (B[j * K + k] > 0) last = k;
    return last;
}

}  // namespace

extern "C" d2moe_status d2moe_plan_load_order(int32_t n_experts, int32_t n_bits, const int32_t* B, int32_t policy,
                                              d2moe_plan_item* queue, int32_t capacity, int32_t* n_items) {
    if (!B || !queue || !n_items) return D2MOE_ERR_NULL;
    if (n_experts <= 0 || n_bits <= 0 || n_bits > 8 || (policy != D2MOE_PLAN_HEBF && policy != D2MOE_PLAN_BY_ID))
        return D2MOE_ERR_CONFIG;
    for (long long i = 0; i < (long long)n_experts * n_bits; ++i)
        if (B[i] < 0) return D2MOE_ERR_SHAPE;
    std::vector<int> last(n_experts), head(n_experts, 0);
    long long total = 0;
    for (int j = 0; j < n_experts; ++j) { last[j] = last_requested(B, n_bits, j); total += last[j] + 1; }
    if (total > capacity) return D2MOE_ERR_WORKSPACE;
    int n = 0;
    if (policy == D2MOE_PLAN_BY_ID) {
        for (int j = 0; j < n_experts; ++j)
            for (int k = 0; k <= last[j]; ++k) queue[n++] = d2moe_plan_item{j, k};
    } else {
        while (n < total) {
            int best = -1;
            long long best_f = -1;
            for (int j = 0; j < n_experts; ++j) {           // ascending id: the first of equal frequencies wins
                if (head[j] > last[j]) continue;
                const long long f = reuse_count(B, n_bits, j, head[j]);
                if (f > best_f) { best_f = f; best = j; }
            }
            queue[n++] = d2moe_plan_item{best, head[best]};
            ++head[best];
        }
    }
    *n_items = n;
    return D2MOE_OK;
}

extern "C" d2moe_status d2moe_plan_simulate(int32_t n_experts, int32_t n_bits, const int32_t* B,
                                            const d2moe_plan_item* queue, int32_t n_items, const double* t_io,
                                            const double* t_comp, double* makespan, double* wait) {
    if (!B || !queue || !t_io || !t_comp || !makespan) return D2MOE_ERR_NULL;
    if (n_experts <= 0 || n_bits <= 0 || n_bits > 8 || n_items < 0) return D2MOE_ERR_CONFIG;
    std::vector<int> next(n_experts, 0);                     // next segment each expert may load (constraint 6b)
    double load_end = 0.0, comp_end = 0.0, w = 0.0;
    for (int s = 0; s < n_items; ++s) {
        const int j = queue[s].expert, k = queue[s].segment;
        if (j < 0 || j >= n_experts || k < 0 || k >= n_bits || k != next[j]) return D2MOE_ERR_SHAPE;
        ++next[j];
        load_end += t_io[k];
        const int n = B[j * n_bits + k];
        if (n > 0) {
            const double start = std::max(comp_end, load_end);  // constraint 6a
            w += start - comp_end;                              // constraint 6c
            comp_end = start + n * t_comp[k];
        }
    }
    *makespan = std::max(comp_end, load_end);
    if (wait) *wait = w;
    return D2MOE_OK;
}

extern "C" d2moe_status d2moe_plan_budget_step(const d2moe_segment* resident, int32_t n_resident,
                                               const d2moe_segment* need, int32_t n_need, int64_t budget,
                                               d2moe_segment* new_resident, int32_t* n_new,
                                               d2moe_segment* loads, int32_t* n_loads,
                                               d2moe_segment* evictions, int32_t* n_evictions, int32_t capacity) {
    if ((n_resident > 0 && !resident) || (n_need > 0 && !need) || !new_resident || !n_new || !loads || !n_loads ||
        !evictions || !n_evictions)
        return D2MOE_ERR_NULL;
    if (n_resident < 0 || n_need < 0 || budget < 0) return D2MOE_ERR_CONFIG;
    auto same = [](const d2moe_segment& a, const d2moe_segment& b) {
        return a.layer == b.layer && a.expert == b.expert && a.segment == b.segment;
    };
    auto in = [&](const d2moe_segment& x, const d2moe_segment* v, int n) {
        for (int i = 0; i < n; ++i)
            if (same(x, v[i])) return true;
        return false;
    };
    std::vector<d2moe_segment> ld, ev;
    long long used = 0, want = 0;
    for (int i = 0; i < n_resident; ++i) used += resident[i].bytes;
    for (int i = 0; i < n_need; ++i)
        if (!in(need[i], resident, n_resident)) { ld.push_back(need[i]); want += need[i].bytes; }
    if (used + want > budget) {
        std::vector<d2moe_segment> victims;
        for (int i = 0; i < n_resident; ++i)
            if (!in(resident[i], need, n_need)) victims.push_back(resident[i]);
        // highest width first, then the oldest layer, then the lowest expert id
        std::stable_sort(victims.begin(), victims.end(), [](const d2moe_segment& a, const d2moe_segment& b) {
            if (a.segment != b.segment) return a.segment > b.segment;
            if (a.layer != b.layer) return a.layer < b.layer;
            return a.expert < b.expert;
        });
        for (const d2moe_segment& v : victims) {
            if (used + want <= budget) break;
            ev.push_back(v);
            used -= v.bytes;
        }
    }
    if (used + want > budget) return D2MOE_ERR_WORKSPACE;       // the layer's own segments exceed the budget
    const long long n_keep = (long long)n_resident - (long long)ev.size();
    if (n_keep + (long long)ld.size() > capacity || (long long)ld.size() > capacity || (long long)ev.size() > capacity)
        return D2MOE_ERR_WORKSPACE;
    int n = 0;
    for (int i = 0; i < n_resident; ++i)
        if (!in(resident[i], ev.data(), (int)ev.size())) new_resident[n++] = resident[i];
    for (const d2moe_segment& x : ld) new_resident[n++] = x;
    *n_new = n;
    for (size_t i = 0; i < ld.size(); ++i) loads[i] = ld[i];
    for (size_t i = 0; i < ev.size(); ++i) evictions[i] = ev[i];
    *n_loads = (int)ld.size();
    *n_evictions = (int)ev.size();
    return D2MOE_OK;
}
