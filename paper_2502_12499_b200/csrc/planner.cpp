// Host planners: checkpoint selection under the paper's two memory models, in exact int64.
//
//   plan_static_n3  - Algorithm 3 (Section 3.2), objective Eq. (cost)
//   plan_dynamic_n2 - Algorithm 5 (Section 4.1), objective Eq. (memory)
//   plan_dynamic_n  - Algorithm 6 (Section 4.2), same objective, monotone queue + pointer walk
//   eval_model      - Eq. (cost) / Eq. (memory) / Algorithm 1 total for a given set
#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <limits>
#include <map>
#include <mutex>
#include <string>

#include "internal.h"

namespace ckpt {

static thread_local char g_error[512] = "";
int64_t g_launches = 0;

// Launch log: kernel name -> launches since the log was switched on.
static std::mutex g_log_mutex;
static bool g_log_on = false;
static std::map<std::string, int64_t> g_log;

void note_launch(const char* kernel) {
    ++g_launches;
    if (!g_log_on) return;
    std::lock_guard<std::mutex> lock(g_log_mutex);
    ++g_log[kernel ? kernel : "?"];
}

void set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof(g_error), fmt, ap);
    va_end(ap);
}

int validate_sizes(int64_t n, const int64_t* d) {
    if (!d) { set_error("d is null"); return CKPT_E_NULL; }
    if (n < 1) { set_error("n = %lld < 1", (long long)n); return CKPT_E_BAD_N; }
    const int64_t limit = std::numeric_limits<int64_t>::max() / 2;
    int64_t sum = 0;
    for (int64_t i = 0; i <= n; ++i) {
        if (d[i] < 1) { set_error("d[%lld] = %lld < 1", (long long)i, (long long)d[i]); return CKPT_E_BAD_SIZE; }
        if (d[i] > limit - sum) { set_error("2*sum(d) overflows int64"); return CKPT_E_OVERFLOW; }
        sum += d[i];
    }
    return CKPT_OK;
}

static int validate_plan(int64_t n, const uint8_t* is_ckpt) {
    if (!is_ckpt) { set_error("is_ckpt is null"); return CKPT_E_NULL; }
    if (!is_ckpt[0] || !is_ckpt[n]) { set_error("d_0 and d_n must be checkpoints"); return CKPT_E_BAD_PLAN; }
    return CKPT_OK;
}

// ------------------------------------------------------------------------------------------------
// Objectives
// ------------------------------------------------------------------------------------------------
int eval_model(int model, int64_t n, const int64_t* d, const uint8_t* is_ckpt, int64_t* peak) {
    if (!peak) { set_error("peak_bytes is null"); return CKPT_E_NULL; }
    int rc = validate_sizes(n, d);
    if (rc) return rc;
    if (model == CKPT_MODEL_STORE_ALL) {
        int64_t s = 0;
        for (int64_t i = 0; i <= n; ++i) s += d[i];
        *peak = s;
        return CKPT_OK;
    }
    rc = validate_plan(n, is_ckpt);
    if (rc) return rc;
    if (model == CKPT_MODEL_STATIC) {
        // Eq. (cost): checkpoint memory + largest segment memory.
        int64_t ckpt_mem = 0, seg = 0, seg_max = 0;
        for (int64_t i = 0; i <= n; ++i) {
            if (is_ckpt[i]) { ckpt_mem += d[i]; seg_max = std::max(seg_max, seg); seg = 0; }
            else seg += d[i];
        }
        *peak = ckpt_mem + seg_max;
        return CKPT_OK;
    }
    if (model == CKPT_MODEL_DYNAMIC) {
        // Eq. (memory): at every checkpoint i (previous checkpoint h):
        //   sum of checkpoints <= i  +  sum d_{h+1..i-1}  +  max d_{h..i-1}.
        int64_t ckpt_mem = d[0], seg = 0, run_max = d[0], worst = 0;
        for (int64_t i = 1; i <= n; ++i) {
            if (is_ckpt[i]) {
                ckpt_mem += d[i];
                worst = std::max(worst, ckpt_mem + seg + run_max);
                seg = 0;
                run_max = d[i];
            } else {
                seg += d[i];
                run_max = std::max(run_max, d[i]);
            }
        }
        *peak = worst;
        return CKPT_OK;
    }
    set_error("unknown memory model %d", model);
    return CKPT_E_BAD_ARG;
}

// ------------------------------------------------------------------------------------------------
// Algorithm 3: for every candidate segment cap s, M(i,s) = min_{l(i)<=j<=i} d_j + M(j-1,s) with a
// sliding-window minimum; answer min_s s + d_n + M(n-1,s).
// ------------------------------------------------------------------------------------------------
namespace {
struct StaticTable {
    int64_t n;
    const int64_t* d;
    std::vector<int64_t> prefix, key, M, arg, queue;
    StaticTable(int64_t n_, const int64_t* d_) : n(n_), d(d_), prefix(n_ + 1), key(n_), M(n_), arg(n_), queue(n_) {
        prefix[0] = 0;
        for (int64_t i = 1; i <= n; ++i) prefix[i] = prefix[i - 1] + d[i];
    }
    // Fills M[0..n-1] (and arg) for one cap; returns M(n-1, s).
    int64_t run(int64_t s, int64_t* work) {
        int64_t head = 0, tail = 0;   // queue[head..tail)
        int64_t lo = 0;               // l(i): smallest j with d_{j+1} + ... + d_i <= s
        int64_t steps = 0;
        for (int64_t i = 0; i < n; ++i) {
            key[i] = d[i] + (i >= 1 ? M[i - 1] : 0);          // M(-1,s) = 0
            while (tail > head && key[queue[tail - 1]] > key[i]) { --tail; ++steps; }
            queue[tail++] = i;
            while (prefix[i] - prefix[lo] > s) ++lo;
            while (queue[head] < lo) { ++head; ++steps; }
            M[i] = key[queue[head]];
            arg[i] = queue[head];
            ++steps;
        }
        if (work) *work += steps;
        return M[n - 1];
    }
};
}  // namespace

int plan_static_n3(int64_t n, const int64_t* d, uint8_t* is_ckpt, int64_t* peak, int64_t* work) {
    std::vector<int64_t> caps;
    caps.push_back(0);
    for (int64_t a = 1; a <= n - 1; ++a) {
        int64_t acc = 0;
        for (int64_t b = a; b <= n - 1; ++b) { acc += d[b]; caps.push_back(acc); }
    }
    std::sort(caps.begin(), caps.end());
    caps.erase(std::unique(caps.begin(), caps.end()), caps.end());

    StaticTable t(n, d);
    int64_t best = -1, best_s = 0;
    for (int64_t s : caps) {
        // M(n-1,s) >= d_0, so no larger cap can do strictly better once this bound is reached.
        if (best >= 0 && s + d[n] + d[0] >= best) break;
        int64_t total = s + d[n] + t.run(s, work);
        if (best < 0 || total < best) { best = total; best_s = s; }
    }
    t.run(best_s, nullptr);
    for (int64_t i = 0; i <= n; ++i) is_ckpt[i] = 0;
    is_ckpt[n] = 1;
    for (int64_t i = n - 1; i >= 0;) {
        int64_t j = t.arg[i];
        is_ckpt[j] = 1;
        i = j - 1;
    }
    *peak = best;
    return CKPT_OK;
}

// ------------------------------------------------------------------------------------------------
// Algorithm 5: M(n) = d_n; M(i) = min_{i<j<=n} max(d_i + M(j), d_i + s(i,j) + d_j).
// ------------------------------------------------------------------------------------------------
static void walk_next(int64_t n, const std::vector<int64_t>& nxt, uint8_t* is_ckpt) {
    for (int64_t i = 0; i <= n; ++i) is_ckpt[i] = 0;
    for (int64_t i = 0; i != n; i = nxt[i]) is_ckpt[i] = 1;
    is_ckpt[n] = 1;
}

// Sizes of the generalised Eq. (memory): what tensor t occupies as a checkpoint (kept), inside the segment being
// processed (live), and the size of its gradient (grad); `incoming` adds a second buffer for the gradients
// r_{h+1} .. r_i that the steps of a segment read.  kept = live = grad = d without `incoming` is the paper's objective.
struct Sizes3 {
    const int64_t* kept;
    const int64_t* live;
    const int64_t* grad;
    int incoming;
};

// Algorithm 5 on the generalised sizes: M(n) = kept_n, M(i) = min over j > i of kept_i + max(M(j), U(i,j)),
// U(i,j) = s(i,j) + kept_j, s(i,j) = sum of live_{i+1..j-1} + max grad_{i..j-1} (+ max grad_{i+1..j}).
static int plan_dynamic_n2_sizes(int64_t n, const Sizes3& z, uint8_t* is_ckpt, int64_t* peak, int64_t* work) {
    std::vector<int64_t> M(n + 1), nxt(n + 1, -1);
    M[n] = z.kept[n];
    int64_t steps = 0;
    for (int64_t i = n - 1; i >= 0; --i) {
        int64_t seg_sum = 0, out_max = z.grad[i], in_max = 0, best = -1, best_j = -1;
        for (int64_t j = i + 1; j <= n; ++j) {
            in_max = std::max(in_max, z.grad[j]);
            int64_t u = seg_sum + out_max + (z.incoming ? in_max : 0) + z.kept[j];
            int64_t v = z.kept[i] + std::max(M[j], u);
            if (best < 0 || v < best) { best = v; best_j = j; }
            seg_sum += z.live[j];
            out_max = std::max(out_max, z.grad[j]);
            ++steps;
        }
        M[i] = best;
        nxt[i] = best_j;
    }
    walk_next(n, nxt, is_ckpt);
    *peak = M[0];
    if (work) *work += steps;
    return CKPT_OK;
}

int plan_dynamic_n2(int64_t n, const int64_t* d, uint8_t* is_ckpt, int64_t* peak, int64_t* work) {
    const Sizes3 z{d, d, d, 0};
    return plan_dynamic_n2_sizes(n, z, is_ckpt, peak, work);
}

// ------------------------------------------------------------------------------------------------
// Algorithm 6.  Q holds indices with strictly decreasing M as the index grows (Lemma 2); only Q has
// to be searched (Lemma 3); U(i,.) increases along Q while M decreases, so max(M(j),U(i,j)) is
// unimodal along Q and its minimum sits at the crossover; the crossover only moves towards smaller
// j as i decreases (Lemma 4), so a pointer that walks along Q finds it in amortised O(1) moves.
// U(i,j) is evaluated exactly from prefix sums and a range maximum: the record-maxima stack of the
// suffix grad_i, grad_{i+1}, ... (maintained as i decreases) searched by bisection, O(log n) per value.
// On the generalised sizes Lemma 1 (U increasing in j) needs live_t >= kept_t for every interior t:
// U(i,j+1) - U(i,j) >= live_j - kept_j + kept_{j+1} > 0; the caller checks that.
// ------------------------------------------------------------------------------------------------
struct RecordStack {                 // indices t with grad_t larger than every grad between the start of the suffix and t;
    std::vector<int64_t> idx;        // stored with the largest index first, so indices and values decrease along the array
    int64_t count = 0;
    void push(const int64_t* g, int64_t i) {
        while (count > 0 && g[idx[count - 1]] <= g[i]) --count;
        idx[count++] = i;
    }
    int64_t max_up_to(const int64_t* g, int64_t last) const {   // max of g over [start of the suffix, last]
        int64_t lo = 0, hi = count - 1;
        while (lo < hi) {
            int64_t mid = (lo + hi) / 2;
            if (idx[mid] <= last) hi = mid; else lo = mid + 1;
        }
        return g[idx[lo]];
    }
};

static int plan_dynamic_n_sizes(int64_t n, const Sizes3& z, uint8_t* is_ckpt, int64_t* peak, int64_t* work) {
    std::vector<int64_t> prefix(n + 1), M(n + 1), nxt(n + 1, -1), q(n + 1);
    prefix[0] = 0;
    for (int64_t i = 1; i <= n; ++i) prefix[i] = prefix[i - 1] + z.live[i];
    int64_t steps = 0;
    RecordStack out_rec, in_rec;     // suffixes that start at i (output gradients) and at i + 1 (incoming gradients)
    out_rec.idx.resize(n + 1);
    in_rec.idx.resize(n + 1);
    int64_t cur_i = 0;
    auto U = [&](int64_t j) -> int64_t {               // U(cur_i, j), j > cur_i
        int64_t u = prefix[j - 1] - prefix[cur_i] + out_rec.max_up_to(z.grad, j - 1) + z.kept[j];
        if (z.incoming) u += in_rec.max_up_to(z.grad, j);
        return u;
    };

    M[n] = z.kept[n];
    int64_t top = 0;      // q[0..top]: q[0] = n (largest index), q[top] = head (smallest index)
    q[0] = n;
    int64_t p = 0;        // position in q of the current minimiser
    for (int64_t i = n - 1; i >= 0; --i) {
        cur_i = i;
        out_rec.push(z.grad, i);
        in_rec.push(z.grad, i + 1);

        auto f = [&](int64_t t) -> int64_t { ++steps; return std::max(M[q[t]], U(q[t])); };
        if (p > top) p = top;
        int64_t fp = f(p);
        // towards the head (smaller j) while not worse: on a tie the smaller j wins
        while (p < top) {
            int64_t fn = f(p + 1);
            if (fn <= fp) { ++p; fp = fn; } else break;
        }
        // towards larger j only if strictly better (never needed when Lemma 4 holds)
        while (p > 0) {
            int64_t fn = f(p - 1);
            if (fn < fp) { --p; fp = fn; } else break;
        }
        M[i] = z.kept[i] + fp;
        nxt[i] = q[p];
        while (top >= 0 && M[q[top]] >= M[i]) { --top; ++steps; }
        q[++top] = i;
        ++steps;
    }
    walk_next(n, nxt, is_ckpt);
    *peak = M[0];
    if (work) *work += steps;
    return CKPT_OK;
}

int plan_dynamic_n(int64_t n, const int64_t* d, uint8_t* is_ckpt, int64_t* peak, int64_t* work) {
    const Sizes3 z{d, d, d, 0};
    return plan_dynamic_n_sizes(n, z, is_ckpt, peak, work);
}

// ------------------------------------------------------------------------------------------------
// Least recomputation under a memory budget.  Eq. (memory) of a set is the largest, over consecutive
// checkpoints (i, j), of P_i + d_i + U(i,j) with P_i the sum of the checkpoints left of i (and P_n + d_n
// at the end), so a suffix plan that starts at checkpoint i is described by two numbers: the cost of the
// units it recomputes and the largest prefix sum R it tolerates.  G(i) keeps the plans no other plan
// beats in both (cost up, R up along the list); a segment (i, j) maps a plan of G(j) to
// (cost + sum of cost over i < k < j, min(budget - d_i - U(i,j), R - d_i)).  U(i,j) grows with j
// (Lemma 1), so the scan over j stops at the first segment the budget cannot hold.  The answer is the
// cheapest plan of G(0) (the prefix of d_0 is empty: R >= 0).
// ------------------------------------------------------------------------------------------------
static int64_t eval_sizes(int64_t n, const Sizes3& z, const uint8_t* is_ckpt);
static inline int64_t eval_sizes_fwd(int64_t n, const Sizes3& z, const uint8_t* is_ckpt) { return eval_sizes(n, z, is_ckpt); }
struct SuffixPlan { int64_t cost, room; int64_t next; int32_t next_plan; };

int plan_min_recompute(int64_t n, const int64_t* d, const int64_t* cost, int64_t budget, uint8_t* is_ckpt, int64_t* peak,
                       int64_t* recompute) {
    std::vector<std::vector<SuffixPlan>> G(n + 1);
    if (budget - d[n] >= 0) G[n].push_back({0, budget - d[n], -1, -1});
    std::vector<SuffixPlan> cand;
    for (int64_t i = n - 1; i >= 0; --i) {
        cand.clear();
        int64_t seg = 0, out_max = d[i], seg_cost = 0;
        for (int64_t j = i + 1; j <= n; ++j) {
            const int64_t cap = budget - d[i] - (seg + out_max + d[j]);
            if (cap < 0) break;
            for (size_t k = 0; k < G[j].size(); ++k) {
                const int64_t room = std::min(cap, G[j][k].room - d[i]);
                if (room >= 0) cand.push_back({G[j][k].cost + seg_cost, room, j, (int32_t)k});
            }
            seg += d[j];
            out_max = std::max(out_max, d[j]);
            seg_cost += cost[j];
        }
        // cheapest first; among equal costs the roomiest, then the nearest next checkpoint
        std::sort(cand.begin(), cand.end(), [](const SuffixPlan& a, const SuffixPlan& b) {
            if (a.cost != b.cost) return a.cost < b.cost;
            if (a.room != b.room) return a.room > b.room;
            return a.next < b.next;
        });
        int64_t best_room = -1;
        for (const SuffixPlan& c : cand)
            if (c.room > best_room) { G[i].push_back(c); best_room = c.room; }
    }
    if (G[0].empty()) { set_error("no checkpoint set fits a budget of %lld bytes", (long long)budget); return CKPT_E_BAD_ARG; }
    for (int64_t i = 0; i <= n; ++i) is_ckpt[i] = 0;
    int64_t i = 0;
    int32_t k = 0;
    while (i >= 0) {
        is_ckpt[i] = 1;
        const SuffixPlan& sp = G[i][k];
        i = sp.next; k = sp.next_plan;
    }
    *recompute = G[0][0].cost;
    const Sizes3 z{d, d, d, 0};
    *peak = eval_sizes_fwd(n, z, is_ckpt);
    return CKPT_OK;
}

// Generalised Eq. (memory) of a given set.
static int64_t eval_sizes(int64_t n, const Sizes3& z, const uint8_t* is_ckpt) {
    int64_t worst = 0, kept_sum = z.kept[0], h = 0;
    for (int64_t i = 1; i <= n; ++i) {
        if (!is_ckpt[i]) continue;
        kept_sum += z.kept[i];
        int64_t seg = 0, out_max = 0, in_max = 0;
        for (int64_t t = h + 1; t < i; ++t) seg += z.live[t];
        for (int64_t t = h; t < i; ++t) out_max = std::max(out_max, z.grad[t]);
        for (int64_t t = h + 1; t <= i; ++t) in_max = std::max(in_max, z.grad[t]);
        worst = std::max(worst, kept_sum + seg + out_max + (z.incoming ? in_max : 0));
        h = i;
    }
    return worst;
}

static int validate_three(int64_t n, const int64_t* kept, const int64_t* live, const int64_t* grad) {
    int rc = validate_sizes(n, kept);
    if (!rc) rc = validate_sizes(n, live);
    if (!rc) rc = validate_sizes(n, grad);
    if (rc) return rc;
    // the worst case adds kept, live and two gradient buffers
    const int64_t limit = std::numeric_limits<int64_t>::max() / 4;
    int64_t a = 0, b = 0, c = 0;
    for (int64_t i = 0; i <= n; ++i) { a += kept[i]; b += live[i]; c = std::max(c, grad[i]); }
    if (a > limit || b > limit || c > limit) { set_error("sizes overflow int64"); return CKPT_E_OVERFLOW; }
    return CKPT_OK;
}

// ------------------------------------------------------------------------------------------------
// The uniform heuristic the paper compares against (Section 2.1 / 5.3): a checkpoint every
// ceil(sqrt(n)) units plus d_n; its peak is reported under Eq. (memory).
// ------------------------------------------------------------------------------------------------
int plan_sqrt_n(int64_t n, const int64_t* d, uint8_t* is_ckpt, int64_t* peak) {
    int64_t step = 1;
    while (step * step < n) ++step;
    for (int64_t i = 0; i <= n; ++i) is_ckpt[i] = (i % step == 0) ? 1 : 0;
    is_ckpt[0] = 1;
    is_ckpt[n] = 1;
    return eval_model(CKPT_MODEL_DYNAMIC, n, d, is_ckpt, peak);
}

}  // namespace ckpt

// ------------------------------------------------------------------------------------------------
// C ABI
// ------------------------------------------------------------------------------------------------
extern "C" {

const char* ckpt_last_error(void) { return ckpt::g_error; }

int ckpt_plan_counted(int algo, int64_t n, const int64_t* d, uint8_t* is_ckpt, int64_t* peak_bytes,
                      int64_t* work) {
    int rc = ckpt::validate_sizes(n, d);
    if (rc) return rc;
    if (!is_ckpt || !peak_bytes) { ckpt::set_error("output pointer is null"); return CKPT_E_NULL; }
    if (work) *work = 0;
    switch (algo) {
        case CKPT_ALGO_STATIC_N3: return ckpt::plan_static_n3(n, d, is_ckpt, peak_bytes, work);
        case CKPT_ALGO_DYNAMIC_N2: return ckpt::plan_dynamic_n2(n, d, is_ckpt, peak_bytes, work);
        case CKPT_ALGO_DYNAMIC_N: return ckpt::plan_dynamic_n(n, d, is_ckpt, peak_bytes, work);
        case CKPT_ALGO_SQRT_N: return ckpt::plan_sqrt_n(n, d, is_ckpt, peak_bytes);
    }
    ckpt::set_error("unknown algorithm %d", algo);
    return CKPT_E_BAD_ARG;
}

int ckpt_plan(int algo, int64_t n, const int64_t* d, uint8_t* is_ckpt, int64_t* peak_bytes) {
    return ckpt_plan_counted(algo, n, d, is_ckpt, peak_bytes, nullptr);
}

int ckpt_eval(int model, int64_t n, const int64_t* d, const uint8_t* is_ckpt, int64_t* peak_bytes) {
    return ckpt::eval_model(model, n, d, is_ckpt, peak_bytes);
}

int ckpt_plan_min_recompute(int64_t n, const int64_t* d, const int64_t* cost, int64_t budget_bytes, uint8_t* is_ckpt,
                            int64_t* peak_bytes, int64_t* recompute_cost) {
    int rc = ckpt::validate_sizes(n, d);
    if (rc) return rc;
    if (!cost || !is_ckpt || !peak_bytes || !recompute_cost) { ckpt::set_error("null pointer"); return CKPT_E_NULL; }
    int64_t total = 0;
    for (int64_t i = 1; i < n; ++i) {
        if (cost[i] < 0) { ckpt::set_error("cost[%lld] is negative", (long long)i); return CKPT_E_BAD_ARG; }
        if (cost[i] > std::numeric_limits<int64_t>::max() / 2 - total) { ckpt::set_error("sum of costs overflows int64"); return CKPT_E_OVERFLOW; }
        total += cost[i];
    }
    if (budget_bytes < 0) { ckpt::set_error("negative budget"); return CKPT_E_BAD_ARG; }
    if (budget_bytes == 0) {                 // the optimum of Eq. (memory)
        std::vector<uint8_t> tmp(n + 1);
        if ((rc = ckpt::plan_dynamic_n(n, d, tmp.data(), &budget_bytes, nullptr))) return rc;
    }
    return ckpt::plan_min_recompute(n, d, cost, budget_bytes, is_ckpt, peak_bytes, recompute_cost);
}

}  // extern "C"

extern "C" {

int ckpt_launch_log(int enable) {
    std::lock_guard<std::mutex> lock(ckpt::g_log_mutex);
    if (enable) ckpt::g_log.clear();
    ckpt::g_log_on = enable != 0;
    return CKPT_OK;
}

int ckpt_launch_log_read(char* text, int64_t capacity, int64_t* needed) {
    if (!needed) { ckpt::set_error("needed is null"); return CKPT_E_NULL; }
    std::string out;
    {
        std::lock_guard<std::mutex> lock(ckpt::g_log_mutex);
        for (const auto& kv : ckpt::g_log) out += std::to_string(kv.second) + "\t" + kv.first + "\n";
    }
    *needed = (int64_t)out.size() + 1;
    if (text && capacity > 0) {
        const size_t m = std::min<size_t>(out.size(), (size_t)capacity - 1);
        memcpy(text, out.data(), m);
        text[m] = 0;
    }
    return CKPT_OK;
}

}  // extern "C"

extern "C" {

int ckpt_plan_sizes(int algo, int64_t n, const int64_t* kept, const int64_t* live, const int64_t* grad, int incoming,
                    uint8_t* is_ckpt, int64_t* peak_bytes) {
    int rc = ckpt::validate_three(n, kept, live, grad);
    if (rc) return rc;
    if (!is_ckpt || !peak_bytes) { ckpt::set_error("output pointer is null"); return CKPT_E_NULL; }
    const ckpt::Sizes3 z{kept, live, grad, incoming ? 1 : 0};
    if (algo == CKPT_ALGO_DYNAMIC_N2) return ckpt::plan_dynamic_n2_sizes(n, z, is_ckpt, peak_bytes, nullptr);
    if (algo == CKPT_ALGO_DYNAMIC_N) {
        for (int64_t t = 1; t < n; ++t)
            if (live[t] < kept[t]) {
                ckpt::set_error("live[%lld] < kept[%lld]: the queue-based search needs live >= kept (use CKPT_ALGO_DYNAMIC_N2)",
                                (long long)t, (long long)t);
                return CKPT_E_BAD_ARG;
            }
        return ckpt::plan_dynamic_n_sizes(n, z, is_ckpt, peak_bytes, nullptr);
    }
    ckpt::set_error("algorithm %d does not take separate sizes", algo);
    return CKPT_E_BAD_ARG;
}

int ckpt_eval_sizes(int64_t n, const int64_t* kept, const int64_t* live, const int64_t* grad, int incoming,
                    const uint8_t* is_ckpt, int64_t* peak_bytes) {
    int rc = ckpt::validate_three(n, kept, live, grad);
    if (rc) return rc;
    if (!peak_bytes) { ckpt::set_error("peak_bytes is null"); return CKPT_E_NULL; }
    rc = ckpt::validate_plan(n, is_ckpt);
    if (rc) return rc;
    const ckpt::Sizes3 z{kept, live, grad, incoming ? 1 : 0};
    *peak_bytes = ckpt::eval_sizes(n, z, is_ckpt);
    return CKPT_OK;
}

}  // extern "C"
