// Parallelism planning (Section 3.3) on the host: Algorithm 1 (allocation of a micro-batch's samples inside a device
// group: memory-aware balancing, then straggler offloading; Eq. (7)-(9)), the latency model of Eq. (4)-(6) with its
// dominant step (Eq. (11)), and Algorithm 2 (dynamic programming over layers, devices and stage count; Eq. (10)).
// Pure host code: it consumes the cost tables that asteroid_stage_profile produces.
#include <algorithm>
#include <cmath>
#include <limits>
#include <map>
#include <tuple>
#include <vector>

#include "../../include/asteroid.h"
#include "kernels.h"

namespace ast {
namespace {

constexpr double INF = std::numeric_limits<double>::infinity();

struct Step {
    bool exec = false;
    int first = 0, last = 0;          // layers (execution steps)
    std::vector<int> group, y;        // devices and their samples
    double ef = 0, eb = 0, ta = 0;
};

struct Pipe {
    bool ok = false;
    double latency = INF;
    int dm = 0;
    std::vector<Step> steps;
};

struct Planner {
    const ast_plan_problem& P;
    explicit Planner(const ast_plan_problem& p) : P(p) {}
    std::map<std::tuple<int, int, int, int, int>, Step> cache;     // (i, j, device range in memory order, K) -> execution step
    std::vector<int> order;

    double tf(int type, int l, int k) const { return P.t_f[((size_t)type * P.L + l) * P.n_bs + k]; }
    double tb(int type, int l, int k) const { return P.t_b[((size_t)type * P.L + l) * P.n_bs + k]; }

    // time at batch size y from the profile: 0 at 0, straight lines between profiled sizes (and from the origin to the
    // first), the last segment continued beyond the largest
    double interp(const double* t, int y) const {
        const int32_t* bs = P.bs;
        const int n = P.n_bs;
        if (y <= 0) return 0.0;
        if (y <= bs[0]) return t[0] * y / bs[0];
        for (int k = 1; k < n; ++k)
            if (y <= bs[k]) return t[k - 1] + (t[k] - t[k - 1]) * (y - bs[k - 1]) / (bs[k] - bs[k - 1]);
        if (n == 1) return t[0] * y / bs[0];
        return t[n - 1] + (t[n - 1] - t[n - 2]) * (y - bs[n - 1]) / (bs[n - 1] - bs[n - 2]);
    }
    void stage_time(int type, int i, int j, int y, double* f, double* b) const {
        double sf = 0.0, sb = 0.0;
        for (int l = i; l <= j; ++l) {
            sf += interp(&P.t_f[((size_t)type * P.L + l) * P.n_bs], y);
            sb += interp(&P.t_b[((size_t)type * P.L + l) * P.n_bs], y);
        }
        *f = sf;
        *b = sb;
    }
    // Eq. (3): largest y with MOD + OPT + K * ACT(y) <= budget; -1 if the model alone does not fit
    long max_batch(double budget, int i, int j, int k_p) const {
        double w = 0.0, act = 0.0;
        for (int l = i; l <= j; ++l) w += P.w[l];
        for (int l = i; l <= j; ++l) act += P.act[l];
        const double fixed = (P.mod_factor + P.opt_factor) * w;
        if (budget < fixed) return -1;
        if (act <= 0) return 1000000000L;
        return (long)std::floor((budget - fixed) / (k_p * act));
    }

    // Algorithm 1.  false: the micro-batch does not fit the group.
    bool allocate(const std::vector<int>& group, int i, int j, int k_p, std::vector<int>& y_out, double* ef, double* eb) const {
        const int n = (int)group.size();
        std::vector<long> cap(n), y(n, 0);
        std::vector<double> v(n);
        for (int q = 0; q < n; ++q) {
            cap[q] = max_batch(P.dev_mem[group[q]], i, j, k_p);
            if (cap[q] < 0) return false;
        }
        for (int q = 0; q < n; ++q) {            // Eq. (9)
            double f, b;
            stage_time(P.dev_type[group[q]], i, j, P.B, &f, &b);
            v[q] = f + b > 0 ? 1.0 / (f + b) : INF;
        }
        // phase 1: MemoryAwareBalancing, written as the loop its tail recursion is
        std::vector<int> G(n);
        for (int q = 0; q < n; ++q) G[q] = q;
        long beta = P.B;
        while (beta != 0) {
            if (G.empty()) return false;
            double vs = 0.0;
            for (int q : G) vs += v[q];
            long given = 0;
            for (int q : G) {
                long share = vs < INF ? (long)std::floor(v[q] / vs * (double)beta) : beta / (long)G.size();
                long take = std::min(share, cap[q] - y[q]);
                y[q] += take;
                given += take;
            }
            long left = beta - given;
            if (given == 0) {                    // all shares rounded down to zero: the fastest device with memory takes one sample
                int best = -1;
                for (int q : G)
                    if (cap[q] - y[q] > 0 && (best < 0 || v[q] > v[best])) best = q;
                if (best < 0) return false;
                y[best] += 1;
                left -= 1;
            }
            std::vector<int> G2;
            for (int q : G)
                if (cap[q] - y[q] > 0) G2.push_back(q);
            G.swap(G2);
            beta = left;
        }
        auto lat = [&](int q) {
            double f, b;
            stage_time(P.dev_type[group[q]], i, j, (int)y[q], &f, &b);
            return f + b;
        };
        // phase 2: StragglerWorkloadOffloading
        while (true) {
            std::vector<int> ord(n);
            std::vector<double> lt(n);
            for (int q = 0; q < n; ++q) {
                ord[q] = q;
                lt[q] = lat(q);
            }
            std::stable_sort(ord.begin(), ord.end(), [&](int a, int b) { return lt[a] < lt[b] || (lt[a] == lt[b] && group[a] < group[b]); });
            const int straggler = ord[n - 1];
            const double old = lt[straggler];
            int to = -1;
            long moved = 0;
            for (int r = 0; r + 1 < n; ++r) {    // fastest first
                const int q = ord[r];
                const long cnt = std::min<long>(P.block, y[straggler]);
                if (cnt > 0 && cap[q] - y[q] >= cnt) {
                    y[straggler] -= cnt;
                    y[q] += cnt;
                    to = q;
                    moved = cnt;
                    break;
                }
            }
            if (to < 0) break;
            double nw = 0.0;
            for (int q = 0; q < n; ++q) nw = std::max(nw, lat(q));
            if (!(nw < old)) {                   // no faster: take the transfer back and stop
                y[to] -= moved;
                y[straggler] += moved;
                break;
            }
        }
        double mf = 0.0, mb = 0.0;
        y_out.resize(n);
        for (int q = 0; q < n; ++q) {
            double f, b;
            stage_time(P.dev_type[group[q]], i, j, (int)y[q], &f, &b);
            mf = std::max(mf, f);
            mb = std::max(mb, b);
            y_out[q] = (int)y[q];
        }
        *ef = mf;
        *eb = mb;
        return true;
    }

    double allreduce_time(const std::vector<int>& group, int i, int j) const {      // Eq. (5)
        if (group.size() < 2) return 0.0;
        double w = 0.0;
        for (int l = i; l <= j; ++l) w += P.w[l];
        double bw = INF;
        for (int a : group)
            for (int b : group)
                if (a != b) bw = std::min(bw, P.bw[(size_t)a * P.N + b]);
        return 2.0 * ((double)group.size() - 1) * w / ((double)group.size() * bw);
    }

    // execution step of layers i..j on devices order[lo, hi); ok == false if the micro-batch does not fit
    const Step* exec_step(int lo, int hi, int i, int j, int k_p) {
        auto key = std::make_tuple(i, j, lo, hi, k_p);
        auto it = cache.find(key);
        if (it == cache.end()) {
            Step s;
            s.exec = true;
            s.first = i;
            s.last = j;
            s.group.assign(order.begin() + lo, order.begin() + hi);
            bool ok = allocate(s.group, i, j, k_p, s.y, &s.ef, &s.eb);
            if (ok) s.ta = allreduce_time(s.group, i, j);
            else s.group.clear();                // marks "does not fit"
            it = cache.emplace(key, std::move(s)).first;
        }
        return it->second.group.empty() ? nullptr : &it->second;
    }

    static double round_latency(const std::vector<Step>& st, int M, int dm) {       // Eq. (4)-(6)
        double worst = 0.0;
        const int S = (int)st.size();
        for (int s = 0; s < S; ++s) {
            double tw = 0.0;
            for (int i = 0; i < s; ++i) tw += st[i].ef;
            double te = M * (st[dm].ef + st[dm].eb);
            if (s < dm) {
                double add = 0.0;
                for (int i = s; i < dm; ++i) add += st[i].ef + st[i].eb;
                te += add;
            } else {
                double sub = 0.0;
                for (int i = dm; i < s; ++i) sub += st[i].ef + st[i].eb;
                te -= sub;
            }
            worst = std::max(worst, tw + te + st[s].ta);
        }
        return worst;
    }

    Pipe run() {
        const int L = P.L, N = P.N, M = P.M;
        order.resize(N);
        for (int d = 0; d < N; ++d) order[d] = d;
        std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return P.dev_mem[a] > P.dev_mem[b] || (P.dev_mem[a] == P.dev_mem[b] && a < b); });
        const int PM = std::min(L, N);
        // Q[(p-1)][n][l]
        std::vector<Pipe> Q((size_t)PM * (N + 1) * (L + 1));
        auto q = [&](int l, int n, int p) -> Pipe& { return Q[((size_t)(p - 1) * (N + 1) + n) * (L + 1) + l]; };
        for (int p = 1; p <= PM; ++p) {
            const int k_p = 2 * p - 1;           // the new head stage is the p-th from the end of the pipeline
            for (int n = 1; n <= N; ++n)
                for (int l = 1; l <= L; ++l) {
                    Pipe best;
                    for (int n2 = 0; n2 < n; ++n2)
                        for (int l2 = 0; l2 < l; ++l2) {
                            const Pipe* sub = nullptr;
                            if (p == 1) {
                                if (n2 != 0 || l2 != 0) continue;
                            } else {
                                if (n2 == 0 || l2 == 0) continue;
                                sub = &q(l2, n2, p - 1);
                                if (!sub->ok) continue;
                            }
                            const int i = L - l, j = L - l2 - 1;
                            const Step* ne = exec_step(N - n, N - n2, i, j, k_p);
                            if (!ne) continue;
                            std::vector<Step> steps;
                            int dm = 0;
                            steps.push_back(*ne);
                            if (sub) {
                                Step nc;
                                double bw = INF;
                                for (int a : ne->group)
                                    for (int b : sub->steps[0].group) bw = std::min(bw, P.bw[(size_t)a * N + b]);
                                nc.ef = nc.eb = P.B * P.a[j] / bw;
                                steps.push_back(nc);
                                steps.insert(steps.end(), sub->steps.begin(), sub->steps.end());
                                // Eq. (11): old dominant step (two places further back), new execution step, new communication step
                                const int od = sub->dm + 2;
                                double pre = 0.0;
                                for (int s = 0; s < od; ++s) pre += steps[s].ef + steps[s].eb;
                                const double va = M * (steps[od].ef + steps[od].eb) + pre;
                                const double vb = M * (ne->ef + ne->eb);
                                const double vc = M * (nc.ef + nc.eb) + (ne->ef + ne->eb);
                                double top = vb;
                                if (vc > top) {
                                    dm = 1;
                                    top = vc;
                                }
                                if (va > top) {
                                    dm = od;
                                    top = va;
                                }
                            }
                            const double lat = round_latency(steps, M, dm);
                            if (!best.ok || lat < best.latency) {
                                best.ok = true;
                                best.latency = lat;
                                best.dm = dm;
                                best.steps.swap(steps);
                            }
                        }
                    q(l, n, p) = std::move(best);
                }
        }
        Pipe out;
        for (int p = 1; p <= PM; ++p) {
            const Pipe& c = q(L, N, p);
            if (c.ok && (!out.ok || c.latency < out.latency)) out = c;
        }
        return out;
    }
};

}  // namespace
}  // namespace ast

extern "C" int asteroid_plan(const ast_plan_problem* p, ast_plan_result* out) {
    using namespace ast;
    if (!p || !out) return report_error(AST_ERR_ARG, "asteroid_plan: null argument");
    if (p->L < 1 || p->N < 1 || p->N > AST_PLAN_MAX_DEVICES || p->n_types < 1 || p->n_bs < 1 || p->B < 1 || p->M < 1 || p->block < 1)
        return report_error(AST_ERR_ARG, "asteroid_plan: sizes must be positive and at most 64 devices");
    if (!p->bs || !p->t_f || !p->t_b || !p->a || !p->w || !p->act || !p->dev_type || !p->dev_mem || !p->bw)
        return report_error(AST_ERR_ARG, "asteroid_plan: null table");
    for (int k = 0; k < p->n_bs; ++k)
        if (p->bs[k] < 1 || (k > 0 && p->bs[k] <= p->bs[k - 1])) return report_error(AST_ERR_ARG, "asteroid_plan: batch sizes must be positive and ascending");
    for (int d = 0; d < p->N; ++d)
        if (p->dev_type[d] < 0 || p->dev_type[d] >= p->n_types) return report_error(AST_ERR_ARG, "asteroid_plan: device type out of range");
    Planner pl(*p);
    Pipe r = pl.run();
    *out = ast_plan_result{};
    out->latency_ms = r.ok ? r.latency : std::numeric_limits<double>::infinity();
    if (!r.ok) return AST_OK;                    // nothing fits: n_stages = 0, infinite latency
    out->dominant_step = r.dm;
    out->n_steps = (int32_t)r.steps.size();
    int s = 0, dpos = 0;
    for (const Step& st : r.steps) {
        if (!st.exec) continue;
        out->first_layer[s] = st.first;
        out->last_layer[s] = st.last;
        out->dev_begin[s] = dpos;
        for (size_t q = 0; q < st.group.size(); ++q) {
            out->devices[dpos] = st.group[q];
            out->samples[dpos] = st.y[q];
            ++dpos;
        }
        out->e_f_ms[s] = st.ef;
        out->e_b_ms[s] = st.eb;
        out->t_a_ms[s] = st.ta;
        ++s;
    }
    out->dev_begin[s] = dpos;
    out->n_stages = s;
    return AST_OK;
}
