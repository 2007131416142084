// Type-directed synthesis of a redistribution (host only).
//
// Follows Section 7 of the paper: the mesh is decomposed into prime-sized axes (Principle 1,
// Section 3); a shortest path is searched in the graph whose nodes are weak types -- identified by
// their local type alone (Section 7.2) -- and whose edges are the multi-axes weak collectives
// dynslice / alltoall / allgather weighted by the cost model (figure "Costs derived from the total
// number of bytes communicated"); the path is lowered to device-map collectives (Lowering Lemma,
// Section 6.1), concretising axes with a bias towards the target type (Section 7.3); at most one
// allpermute is appended and moved before any trailing allgathers (Section 7.3).
#include <algorithm>
#include <cstring>
#include <limits>
#include <map>
#include <queue>

#include "plan.hpp"

namespace redist {

namespace {

std::vector<i64> factorize(i64 k)
{
    std::vector<i64> f;
    for (i64 p = 2; p * p <= k; ++p)
        while (k % p == 0) {
            f.push_back(p);
            k /= p;
        }
    if (k > 1) f.push_back(k);
    return f;   // ascending
}

i64 tile_index(const Plan &p, const ConcreteState &s, int d, int k)
{
    // D[[c{x, xs}n]](i) / c = i_x + |x| * (...): mixed radix over the axis list, first = fastest
    i64 t = 0, stride = 1;
    for (int a : s.ax[k]) {
        t += s.lc[d][a] * stride;
        stride *= p.primes[a].size;
    }
    return t;
}

i64 axes_product(const Plan &p, const std::vector<int> &ax)
{
    i64 n = 1;
    for (int a : ax) n *= p.primes[a].size;
    return n;
}

// ------------------------------------------------------------------------------ weak graph search

struct WeakStep {
    int kind, i, j;
    std::vector<int> e;   // exponent of every distinct mesh prime in the factor moved
    i64 factor;
};

struct Search {
    const Plan &p;
    std::vector<i64> P;            // distinct primes of the mesh, ascending
    std::vector<int> mesh_cnt;     // how many mesh axes have that prime size
    int r, np;
    i64 M;                         // max(localsize src, localsize dst)
    std::vector<int> tgt_exps;     // target exponents [r*np]

    bool allow_over = false;       // ignore REDIST_NO_OVERPARTITION (fallback when it leaves no path)
    i64 lat;                       // per-step latency, in elements, added to every edge weight: the cost
                                   // model of Section 6.2 counts bytes only, while small transfers are bound
                                   // by the latency of each collective (Section 8, third research question);
                                   // 0 = the paper's weights

    explicit Search(const Plan &plan) : p(plan), r(plan.rank), np(0), M(0), lat(std::max<i64>(0, plan.tuning.step_latency)) {}

    i64 pow_of(const std::vector<int> &e) const
    {
        i64 m = 1;
        for (int q = 0; q < np; ++q)
            for (int t = 0; t < e[q]; ++t) m *= P[q];
        return m;
    }
    i64 shard_factor(const std::vector<uint8_t> &key, int k) const
    {
        i64 f = 1;
        for (int q = 0; q < np; ++q)
            for (int t = 0; t < key[k * np + q]; ++t) f *= P[q];
        return f;
    }
    i64 localsize(const std::vector<uint8_t> &key) const
    {
        i64 L = 1;
        for (int k = 0; k < r; ++k) L *= p.global_shape[k] / shard_factor(key, k);
        return L;
    }
    std::vector<uint8_t> key_of(const std::vector<std::vector<int>> &pax, int phase) const
    {
        std::vector<uint8_t> key(r * np + 1, 0);
        for (int k = 0; k < r; ++k)
            for (int a : pax[k]) {
                int q = int(std::lower_bound(P.begin(), P.end(), p.primes[a].size) - P.begin());
                key[k * np + q]++;
            }
        key[r * np] = uint8_t(phase);
        return key;
    }

    // all non-zero exponent vectors below caps
    template <class F>
    void for_each_factor(const std::vector<int> &caps, F f) const
    {
        std::vector<int> e(np, 0);
        while (true) {
            int q = 0;
            while (q < np && e[q] == caps[q]) e[q++] = 0;
            if (q == np) return;
            e[q]++;
            f(e);
        }
    }

    // Every weak collective that applies to the weak type `key` (its last entry is the phase of the
    // normal form: 0 = dynslices still allowed, 1 = alltoalls, 2 = allgathers only), reported as
    // relax(successor, weight, step).
    template <class R>
    void expand(const std::vector<uint8_t> &key, bool no_over, R relax) const
    {
        using Key = std::vector<uint8_t>;
        const int phase = key[r * np];
        std::vector<i64> c(r);
        i64 L = 1;
        std::vector<int> used(np, 0);
        for (int k = 0; k < r; ++k) {
            c[k] = p.global_shape[k] / shard_factor(key, k);
            L *= c[k];
            for (int q = 0; q < np; ++q) used[q] += key[k * np + q];
        }
        // dynslice(i, m): m from unused primes, m | c_i, weight 0 (phase 0 only: normal form)
        if (phase == 0) {
            std::vector<int> caps(np);
            for (int q = 0; q < np; ++q) caps[q] = mesh_cnt[q] - used[q];
            for (int i = 0; i < r; ++i)
                for_each_factor(caps, [&](const std::vector<int> &e) {
                    i64 m = pow_of(e);
                    if (c[i] % m) return;
                    if (no_over)
                        for (int q = 0; q < np; ++q) {
                            if (e[q] == 0) continue;
                            int tgt_used = 0;
                            for (int k = 0; k < r; ++k) tgt_used += tgt_exps[k * np + q];
                            if (key[i * np + q] + e[q] > tgt_exps[i * np + q] || used[q] + e[q] > tgt_used)
                                return;
                        }
                    Key nk = key;
                    for (int q = 0; q < np; ++q) nk[i * np + q] = uint8_t(nk[i * np + q] + e[q]);
                    relax(nk, lat, WeakStep{REDIST_STEP_DYNSLICE, i, -1, e, m});
                });
        }
        // alltoall(i -> j, m): m from the primes on dim i, m | c_j, weight localsize (phases 0, 1)
        if (phase <= 1) {
            for (int i = 0; i < r; ++i) {
                std::vector<int> caps(np);
                for (int q = 0; q < np; ++q) caps[q] = key[i * np + q];
                for (int j = 0; j < r; ++j) {
                    if (j == i) continue;
                    for_each_factor(caps, [&](const std::vector<int> &e) {
                        i64 m = pow_of(e);
                        if (c[j] % m) return;
                        Key nk = key;
                        for (int q = 0; q < np; ++q) {
                            nk[i * np + q] = uint8_t(nk[i * np + q] - e[q]);
                            nk[j * np + q] = uint8_t(nk[j * np + q] + e[q]);
                        }
                        nk[r * np] = 1;
                        relax(nk, L + lat, WeakStep{REDIST_STEP_ALLTOALL, i, j, e, m});
                    });
                }
            }
        }
        // allgather(i, m): m from the primes on dim i, weight = new localsize <= M
        for (int i = 0; i < r; ++i) {
            std::vector<int> caps(np);
            for (int q = 0; q < np; ++q) caps[q] = key[i * np + q];
            for_each_factor(caps, [&](const std::vector<int> &e) {
                i64 m = pow_of(e);
                if (L > M / m) return;   // L * m <= M, overflow-safe
                Key nk = key;
                for (int q = 0; q < np; ++q) nk[i * np + q] = uint8_t(nk[i * np + q] - e[q]);
                nk[r * np] = 2;
                relax(nk, L * m + lat, WeakStep{REDIST_STEP_ALLGATHER, i, -1, e, m});
            });
        }
    }

    // All shortest paths (minimal cost, then minimal number of steps), up to `max_paths` of them:
    // the weak graph cannot tell them apart, the lowering can (one may need no final permutation).
    bool run(std::vector<std::vector<WeakStep>> &paths, size_t max_paths)
    {
        for (const PrimeAxis &a : p.primes) {
            auto it = std::lower_bound(P.begin(), P.end(), a.size);
            if (it == P.end() || *it != a.size) P.insert(it, a.size);
        }
        np = int(P.size());
        mesh_cnt.assign(np, 0);
        for (const PrimeAxis &a : p.primes) mesh_cnt[std::lower_bound(P.begin(), P.end(), a.size) - P.begin()]++;
        M = std::max(p.local_src, p.local_dst);
        using Key = std::vector<uint8_t>;
        Key start = key_of(p.src_pax, 0);
        Key goal = key_of(p.dst_pax, 0);
        tgt_exps.assign(goal.begin(), goal.end() - 1);
        const bool no_over = (p.flags & REDIST_NO_OVERPARTITION) != 0 && !allow_over;

        struct Info {
            i64 cost;
            int nsteps;
            std::vector<std::pair<Key, WeakStep>> preds;   // every tight predecessor
            bool done;
        };
        std::map<Key, Info> info;
        struct QE {
            i64 cost;
            int nsteps;
            uint64_t seq;
            Key key;
            bool operator>(const QE &o) const
            {
                if (cost != o.cost) return cost > o.cost;
                if (nsteps != o.nsteps) return nsteps > o.nsteps;
                return seq > o.seq;
            }
        };
        std::priority_queue<QE, std::vector<QE>, std::greater<QE>> pq;
        uint64_t seq = 0;
        info[start] = Info{0, 0, {}, false};
        pq.push(QE{0, 0, seq++, start});
        std::vector<Key> found;
        i64 best_cost = 0;
        int best_steps = 0;
        while (!pq.empty()) {
            QE cur = pq.top();
            pq.pop();
            if (!found.empty() && (cur.cost > best_cost || cur.nsteps > best_steps)) break;
            Info &ci = info[cur.key];
            if (ci.done || ci.cost != cur.cost || ci.nsteps != cur.nsteps) continue;
            ci.done = true;
            if (std::equal(goal.begin(), goal.end() - 1, cur.key.begin())) {
                if (found.empty()) {
                    best_cost = cur.cost;
                    best_steps = cur.nsteps;
                }
                found.push_back(cur.key);
                continue;
            }
            const Key &key = cur.key;
            auto relax = [&](const Key &nk, i64 w, const WeakStep &ws) {
                i64 nc = cur.cost + w;
                int ns = cur.nsteps + 1;
                auto it = info.find(nk);
                if (it != info.end()) {
                    Info &o = it->second;
                    if (o.cost == nc && o.nsteps == ns) {
                        o.preds.push_back({key, ws});
                        return;
                    }
                    if (o.done || o.cost < nc || (o.cost == nc && o.nsteps < ns)) return;
                }
                info[nk] = Info{nc, ns, {{key, ws}}, false};
                pq.push(QE{nc, ns, seq++, nk});
            };
            expand(key, no_over, relax);
        }
        if (found.empty()) return false;
        paths.clear();
        // depth-first enumeration backwards from the goal over tight edges
        struct Frame {
            Key key;
            size_t next;
        };
        for (const Key &gk : found) {
            std::vector<Frame> stack{Frame{gk, 0}};
            std::vector<WeakStep> rev;
            while (!stack.empty() && paths.size() < max_paths) {
                Frame &f = stack.back();
                if (f.key == start) {
                    paths.emplace_back(rev.rbegin(), rev.rend());
                    stack.pop_back();
                    if (!rev.empty()) rev.pop_back();
                    continue;
                }
                const Info &in = info[f.key];
                if (f.next >= in.preds.size()) {
                    stack.pop_back();
                    if (!rev.empty()) rev.pop_back();
                    continue;
                }
                const auto &pr = in.preds[f.next++];
                rev.push_back(pr.second);
                stack.push_back(Frame{pr.first, 0});
            }
        }
        return !paths.empty();
    }
    // Sequences of weak cost strictly below `bound` and of at most `max_steps` steps, those with the
    // cheapest continuation first, at most `max_paths` of them.  The search of Section 7.3 leaves the
    // final permutation out of the edge weights, so a sequence that is not a shortest path can still be
    // the cheaper plan once its permutation -- or the lack of one -- is counted.  Weights and `bound`
    // include the per-step latency.  Call after run().
    void near(i64 bound, int max_steps, size_t max_paths, std::vector<std::vector<WeakStep>> &paths) const
    {
        using Key = std::vector<uint8_t>;
        const bool no_over = (p.flags & REDIST_NO_OVERPARTITION) != 0 && !allow_over;
        const Key start = key_of(p.src_pax, 0);
        struct Edge {
            int to;
            i64 w;
            WeakStep ws;
        };
        const i64 INF = std::numeric_limits<i64>::max();
        std::map<Key, int> id;
        std::vector<Key> keys;
        std::vector<std::vector<Edge>> out;
        std::vector<i64> from_start;
        auto node = [&](const Key &k) {
            auto it = id.find(k);
            if (it != id.end()) return it->second;
            int v = int(keys.size());
            id.emplace(k, v);
            keys.push_back(k);
            out.emplace_back();
            from_start.push_back(INF);
            return v;
        };
        // 1. every weak type within the bound, with its out-edges (Dijkstra order from the source type)
        using QE = std::pair<i64, int>;
        std::priority_queue<QE, std::vector<QE>, std::greater<QE>> pq;
        from_start[node(start)] = 0;
        pq.push({0, 0});
        std::vector<char> expanded;
        while (!pq.empty()) {
            auto [dv, v] = pq.top();
            pq.pop();
            if (expanded.size() < keys.size()) expanded.resize(keys.size(), 0);
            if (expanded[v] || dv != from_start[v]) continue;
            expanded[v] = 1;
            const Key key = keys[v];
            expand(key, no_over, [&](const Key &nk, i64 w, const WeakStep &ws) {
                if (dv + w >= bound) return;
                int u = node(nk);
                out[v].push_back(Edge{u, w, ws});
                if (dv + w < from_start[u]) {
                    from_start[u] = dv + w;
                    pq.push({dv + w, u});
                }
            });
        }
        // 2. cheapest continuation to the target local type, whatever the phase
        const int V = int(keys.size());
        std::vector<std::vector<std::pair<int, i64>>> in(V);
        for (int v = 0; v < V; ++v)
            for (const Edge &e : out[v]) in[e.to].push_back({v, e.w});
        std::vector<i64> to_goal(V, INF);
        std::vector<char> is_goal(V, 0);
        for (int v = 0; v < V; ++v)
            if (std::equal(tgt_exps.begin(), tgt_exps.end(), keys[v].begin())) {
                is_goal[v] = 1;
                to_goal[v] = 0;
                pq.push({0, v});
            }
        while (!pq.empty()) {
            auto [dv, v] = pq.top();
            pq.pop();
            if (dv != to_goal[v]) continue;
            for (auto [u, w] : in[v])
                if (dv + w < to_goal[u]) {
                    to_goal[u] = dv + w;
                    pq.push({dv + w, u});
                }
        }
        for (int v = 0; v < V; ++v)
            std::stable_sort(out[v].begin(), out[v].end(), [&](const Edge &a, const Edge &b) {
                i64 ca = to_goal[a.to] == INF ? INF : a.w + to_goal[a.to];
                i64 cb = to_goal[b.to] == INF ? INF : b.w + to_goal[b.to];
                return ca < cb;
            });
        // 3. depth-first enumeration under the bound (dynslices only add axes and every other step
        //    costs at least one element, so no walk is endless); the visit budget keeps planning fast
        struct Frame {
            int v;
            size_t next;
            i64 cost;
        };
        std::vector<Frame> stack{Frame{0, 0, 0}};
        std::vector<WeakStep> cur;
        size_t visits = 0;
        while (!stack.empty() && paths.size() < max_paths && visits < 20000) {
            Frame &f = stack.back();
            if (f.next == 0 && is_goal[f.v] && !cur.empty()) paths.push_back(cur);
            if (is_goal[f.v] || f.next >= out[f.v].size() || int(stack.size()) > max_steps) {
                stack.pop_back();
                if (!cur.empty()) cur.pop_back();
                continue;
            }
            const Edge &e = out[f.v][f.next++];
            ++visits;
            if (to_goal[e.to] == INF || f.cost + e.w + to_goal[e.to] >= bound) continue;
            cur.push_back(e.ws);
            const i64 nc = f.cost + e.w;
            stack.push_back(Frame{e.to, 0, nc});
        }
    }
};

// ------------------------------------------------------------------------------------- lowering

struct Lowerer {
    const Plan &p;
    const Search &S;
    explicit Lowerer(const Plan &plan, const Search &s) : p(plan), S(s) {}

    int prime_index(int axis) const
    {
        return int(std::lower_bound(S.P.begin(), S.P.end(), p.primes[axis].size) - S.P.begin());
    }
    static int pos_in(const std::vector<int> &list, int a)
    {
        auto it = std::find(list.begin(), list.end(), a);
        return it == list.end() ? -1 : int(it - list.begin());
    }
    bool used_by_target(int a) const
    {
        for (const auto &l : p.dst_pax)
            if (pos_in(l, a) >= 0) return true;
        return false;
    }

    // Pick, for every prime q, e[q] axes of that size among `cands`, best score first.
    struct Scored {
        int cls, sub, axis;
        bool operator<(const Scored &o) const
        {
            if (cls != o.cls) return cls < o.cls;
            if (sub != o.sub) return sub < o.sub;
            return axis < o.axis;
        }
    };
    bool pick(std::vector<Scored> cands, const std::vector<int> &e, std::vector<int> &chosen) const
    {
        std::sort(cands.begin(), cands.end());
        std::vector<int> need = e;
        chosen.clear();
        for (const Scored &s : cands) {
            int q = prime_index(s.axis);
            if (need[q] > 0) {
                need[q]--;
                chosen.push_back(s.axis);
            }
        }
        for (int n : need)
            if (n) return false;
        return true;
    }

    // Order a block that will sit at the minor end of target dimension j: axes the target does not
    // want there first (they have to leave again), then the target's axes in the target's order.
    void order_block(std::vector<int> &block, int j) const
    {
        std::stable_sort(block.begin(), block.end(), [&](int a, int b) {
            int pa = pos_in(p.dst_pax[j], a), pb = pos_in(p.dst_pax[j], b);
            if ((pa < 0) != (pb < 0)) return pa < 0;
            if (pa < 0) return a < b;
            return pa < pb;
        });
    }

    // Low-level rules: bring `block` to the front of dimension k by relabelling devices -- every
    // device keeps its tile index (beta' o phi'^-1 = beta o phi^-1), so no data moves.
    void relabel_to_front(ConcreteState &s, int k, const std::vector<int> &block) const
    {
        std::vector<int> order = block;
        for (int a : s.ax[k])
            if (pos_in(block, a) < 0) order.push_back(a);
        if (order == s.ax[k]) return;
        const int N = p.n_devices;
        for (int d = 0; d < N; ++d) {
            i64 t = tile_index(p, s, d, k);
            for (int a : order) {
                s.lc[d][a] = int(t % p.primes[a].size);
                t /= p.primes[a].size;
            }
        }
        s.ax[k] = order;
    }

    bool lower(const std::vector<WeakStep> &path, std::vector<Step> &steps, ConcreteState &end) const
    {
        ConcreteState cur = p.initial;
        steps.clear();
        for (const WeakStep &w : path) {
            Step st;
            st.kind = w.kind;
            st.dim_i = w.i;
            st.dim_j = w.j;
            st.factor = w.factor;
            st.local_before = localtype_of(p, cur);
            std::vector<Scored> cands;
            if (w.kind == REDIST_STEP_DYNSLICE) {
                std::vector<char> used(p.primes.size(), 0);
                for (const auto &l : cur.ax)
                    for (int a : l) used[a] = 1;
                for (int a = 0; a < int(p.primes.size()); ++a) {
                    if (used[a]) continue;
                    int pos = pos_in(p.dst_pax[w.i], a);
                    if (pos >= 0)
                        cands.push_back({0, -pos, a});
                    else
                        cands.push_back({used_by_target(a) ? 2 : 1, 0, a});
                }
                if (!pick(cands, w.e, st.acting)) return false;
                order_block(st.acting, w.i);
                st.pre = cur;
                std::vector<int> nl = st.acting;
                nl.insert(nl.end(), cur.ax[w.i].begin(), cur.ax[w.i].end());
                cur.ax[w.i] = nl;
            } else if (w.kind == REDIST_STEP_ALLTOALL) {
                for (int a : cur.ax[w.i]) {
                    int pos = pos_in(p.dst_pax[w.j], a);
                    if (pos >= 0)
                        cands.push_back({0, -pos, a});
                    else
                        cands.push_back({pos_in(p.dst_pax[w.i], a) < 0 ? 1 : 2, pos_in(cur.ax[w.i], a), a});
                }
                if (!pick(cands, w.e, st.acting)) return false;
                order_block(st.acting, w.j);
                relabel_to_front(cur, w.i, st.acting);
                st.pre = cur;
                cur.ax[w.i].erase(cur.ax[w.i].begin(), cur.ax[w.i].begin() + st.acting.size());
                std::vector<int> nl = st.acting;
                nl.insert(nl.end(), cur.ax[w.j].begin(), cur.ax[w.j].end());
                cur.ax[w.j] = nl;
            } else {   // allgather
                for (int a : cur.ax[w.i])
                    cands.push_back({pos_in(p.dst_pax[w.i], a) < 0 ? 0 : 1, pos_in(cur.ax[w.i], a), a});
                if (!pick(cands, w.e, st.acting)) return false;
                std::sort(st.acting.begin(), st.acting.end(),
                          [&](int a, int b) { return pos_in(cur.ax[w.i], a) < pos_in(cur.ax[w.i], b); });
                relabel_to_front(cur, w.i, st.acting);
                st.pre = cur;
                cur.ax[w.i].erase(cur.ax[w.i].begin(), cur.ax[w.i].begin() + st.acting.size());
            }
            st.post = cur;
            st.local_after = localtype_of(p, cur);
            steps.push_back(st);
        }
        end = cur;
        return true;
    }
};

bool same_assignment(const Plan &p, const ConcreteState &a, const ConcreteState &b)
{
    for (int d = 0; d < p.n_devices; ++d)
        for (int k = 0; k < p.rank; ++k)
            if (tile_index(p, a, d, k) != tile_index(p, b, d, k)) return false;
    return true;
}

// A bijection on devices that takes assignment `from` to assignment `to` (it exists whenever the
// local and global types agree, Section 5): devices already holding their tile keep it, the others
// are matched in ascending device id.
bool make_permutation(const Plan &p, const ConcreteState &from, const ConcreteState &to,
                      std::vector<int> &source_of)
{
    const int N = p.n_devices;
    Layout lf = layout_of(p, from), lt = layout_of(p, to);
    if (lf.tile != lt.tile) return false;
    source_of.assign(N, -1);
    std::vector<char> taken(N, 0);
    for (int d = 0; d < N; ++d)
        if (lf.tile_of[d] == lt.tile_of[d]) {
            source_of[d] = d;
            taken[d] = 1;
        }
    std::map<int32_t, std::vector<int>> pool;
    for (int d = N - 1; d >= 0; --d)
        if (!taken[d]) pool[lf.tile_of[d]].push_back(d);   // back() = lowest id
    for (int d = 0; d < N; ++d) {
        if (source_of[d] >= 0) continue;
        auto it = pool.find(lt.tile_of[d]);
        if (it == pool.end() || it->second.empty()) return false;
        source_of[d] = it->second.back();
        it->second.pop_back();
    }
    return true;
}

i64 product(const std::vector<i64> &v)
{
    i64 n = 1;
    for (i64 x : v) n *= x;
    return n;
}

}  // namespace

// ---------------------------------------------------------------------------------- public pieces

redist_status check_type(int n_axes, const i64 *mesh, const redist_type *t, std::vector<i64> *tile)
{
    if (!t || t->rank < 1 || t->rank > REDIST_MAX_RANK || !t->global_shape || !t->axes_off) return REDIST_EINVAL;
    if (t->axes_off[0] != 0) return REDIST_EINVAL;
    std::vector<char> used(n_axes, 0);
    tile->assign(t->rank, 0);
    for (int k = 0; k < t->rank; ++k) {
        if (t->global_shape[k] < 1) return REDIST_EINVAL;
        if (t->axes_off[k + 1] < t->axes_off[k]) return REDIST_EINVAL;
        if (t->axes_off[k + 1] > t->axes_off[k] && !t->axes) return REDIST_EINVAL;
    }
    for (int k = 0; k < t->rank; ++k) {
        i64 prod = 1;
        for (int q = t->axes_off[k]; q < t->axes_off[k + 1]; ++q) {
            int a = t->axes[q];
            if (a < 0 || a >= n_axes) return REDIST_EILLFORMED;   // wf-dim: the axis is in the mesh
            if (used[a]) return REDIST_EILLFORMED;                // distinct within / disjoint across dims
            used[a] = 1;
            prod *= mesh[a];
        }
        if (t->global_shape[k] % prod) return REDIST_ENOTDIV;     // wf-dim: c * prod(k_i) = n
        (*tile)[k] = t->global_shape[k] / prod;
    }
    return REDIST_OK;
}

void base_offsets_of(int n_axes, const i64 *mesh, const redist_type *t, const std::vector<i64> &tile, i64 *out)
{
    i64 N = 1;
    for (int a = 0; a < n_axes; ++a) N *= mesh[a];
    std::vector<i64> coord(n_axes > 0 ? n_axes : 1);
    for (i64 d = 0; d < N; ++d) {
        i64 rem = d;
        for (int a = n_axes - 1; a >= 0; --a) {
            coord[a] = rem % mesh[a];
            rem /= mesh[a];
        }
        for (int k = 0; k < t->rank; ++k) {
            // D[[c{x, xs}n]] = c * i_x + D[[(c * |x|){xs}n]]
            i64 c = tile[k], off = 0;
            for (int q = t->axes_off[k]; q < t->axes_off[k + 1]; ++q) {
                off += c * coord[t->axes[q]];
                c *= mesh[t->axes[q]];
            }
            out[d * t->rank + k] = off;
        }
    }
}

std::vector<i64> localtype_of(const Plan &p, const ConcreteState &s)
{
    std::vector<i64> c(p.rank);
    for (int k = 0; k < p.rank; ++k) c[k] = p.global_shape[k] / axes_product(p, s.ax[k]);
    return c;
}

Layout layout_of(const Plan &p, const ConcreteState &s)
{
    Layout l;
    l.tile = localtype_of(p, s);
    l.ntiles.resize(p.rank);
    for (int k = 0; k < p.rank; ++k) l.ntiles[k] = p.global_shape[k] / l.tile[k];
    l.tile_of.resize(p.n_devices);
    for (int d = 0; d < p.n_devices; ++d) {
        i64 lin = 0;
        for (int k = 0; k < p.rank; ++k) lin = lin * l.ntiles[k] + tile_index(p, s, d, k);
        l.tile_of[d] = int32_t(lin);
    }
    return l;
}

redist_status synthesize(Plan &p)
{
    const int N = p.n_devices;
    // 1. prime-factor mesh: axis x:k becomes x1:p1, ..., xm:pm (ascending primes, minor first)
    std::vector<std::vector<int>> prime_of_axis(p.n_mesh_axes);
    p.primes.clear();
    for (int a = 0; a < p.n_mesh_axes; ++a) {
        i64 stride = 1;
        for (i64 f : factorize(p.mesh_shape[a])) {
            prime_of_axis[a].push_back(int(p.primes.size()));
            p.primes.push_back(PrimeAxis{a, f, stride});
            stride *= f;
        }
    }
    auto to_prime = [&](const std::vector<std::vector<int>> &axes) {
        std::vector<std::vector<int>> out(axes.size());
        for (size_t k = 0; k < axes.size(); ++k)
            for (int a : axes[k]) out[k].insert(out[k].end(), prime_of_axis[a].begin(), prime_of_axis[a].end());
        return out;
    };
    p.src_pax = to_prime(p.src_axes);
    p.dst_pax = to_prime(p.dst_axes);
    const int A = int(p.primes.size());
    // canonical device map: the logical coordinates of device d are its own mesh coordinates
    std::vector<std::vector<int>> lc0(N, std::vector<int>(A > 0 ? A : 1, 0));
    for (int d = 0; d < N; ++d) {
        std::vector<i64> coord(p.n_mesh_axes > 0 ? p.n_mesh_axes : 1, 0);
        i64 rem = d;
        for (int a = p.n_mesh_axes - 1; a >= 0; --a) {
            coord[a] = rem % p.mesh_shape[a];
            rem /= p.mesh_shape[a];
        }
        for (int a = 0; a < A; ++a)
            lc0[d][a] = int((coord[p.primes[a].parent] / p.primes[a].parent_stride) % p.primes[a].size);
    }
    p.initial.ax = p.src_pax;
    p.initial.lc = lc0;
    ConcreteState target;
    target.ax = p.dst_pax;
    target.lc = lc0;
    p.local_src = product(localtype_of(p, p.initial));
    p.local_dst = product(localtype_of(p, target));

    // 2. shortest paths over weak types
    Search S(p);
    std::vector<std::vector<WeakStep>> paths;
    if (!S.run(paths, 64)) {
        // the over-partitioning ban may leave no path inside the memory bound: drop it rather than fail
        S.allow_over = true;
        S.P.clear();
        if (!S.run(paths, 64)) return REDIST_EINTERNAL;
    }

    // 3. lowering; the equal-cost shortest paths (e.g. the orders of commuting alltoalls) differ in
    //    where the axes end up: keep the first that reaches the target assignment without a
    //    permutation, otherwise the first that lowers at all
    Lowerer L(p, S);
    std::vector<Step> steps;
    ConcreteState end;
    bool have = false;
    for (const auto &cand : paths) {
        std::vector<Step> st;
        ConcreteState e;
        if (!L.lower(cand, st, e)) continue;
        const bool exact = same_assignment(p, e, target);
        if (!have || exact) {
            steps = st;
            end = e;
            have = true;
        }
        if (exact) break;
    }
    if (!have) return REDIST_EINTERNAL;

    // 4. at most one allpermute, placed before the trailing allgathers; 5. costs and height
    auto finish = [&](std::vector<Step> &steps, ConcreteState &end, i64 &cost, i64 &height) -> redist_status {
        if (!same_assignment(p, end, target)) {
            size_t g0 = steps.size();
            while (g0 > 0 && steps[g0 - 1].kind == REDIST_STEP_ALLGATHER) --g0;
            ConcreteState pre_gather = g0 < steps.size() ? steps[g0].pre : end;
            if (g0 < steps.size()) pre_gather = (g0 == 0) ? p.initial : steps[g0 - 1].post;
            // target type extended by the gathered axes (taken from axes the target leaves unused)
            ConcreteState ext = target;
            std::vector<char> busy(A, 0);
            for (const auto &l : p.dst_pax)
                for (int a : l) busy[a] = 1;
            std::vector<std::vector<int>> blocks;
            std::vector<std::vector<int>> extra(p.rank);
            for (size_t t = g0; t < steps.size(); ++t) {
                std::vector<int> blk;
                for (int a : steps[t].acting) {
                    int pickd = -1;
                    if (!busy[a]) pickd = a;
                    for (int b = 0; b < A && pickd < 0; ++b)
                        if (!busy[b] && p.primes[b].size == p.primes[a].size) pickd = b;
                    if (pickd < 0) return REDIST_EINTERNAL;
                    busy[pickd] = 1;
                    blk.push_back(pickd);
                }
                blocks.push_back(blk);
                extra[steps[t].dim_i].insert(extra[steps[t].dim_i].end(), blk.begin(), blk.end());
            }
            for (int k = 0; k < p.rank; ++k) {
                std::vector<int> nl = extra[k];
                nl.insert(nl.end(), p.dst_pax[k].begin(), p.dst_pax[k].end());
                ext.ax[k] = nl;
            }
            std::vector<Step> tail(steps.begin() + g0, steps.end());
            steps.resize(g0);
            if (!same_assignment(p, pre_gather, ext)) {
                Step pm;
                pm.kind = REDIST_STEP_ALLPERMUTE;
                pm.pre = pre_gather;
                pm.post = ext;
                pm.local_before = localtype_of(p, pre_gather);
                pm.local_after = localtype_of(p, ext);
                if (pm.local_before != pm.local_after) return REDIST_EINTERNAL;
                if (!make_permutation(p, pre_gather, ext, pm.source_of)) return REDIST_EINTERNAL;
                steps.push_back(pm);
            }
            ConcreteState cur = ext;
            for (size_t t = 0; t < tail.size(); ++t) {
                Step g = tail[t];
                g.acting = blocks[t];
                g.pre = cur;
                g.local_before = localtype_of(p, cur);
                const int i = g.dim_i;
                // the block is minor-most in ext by construction
                for (size_t q = 0; q < g.acting.size(); ++q)
                    if (cur.ax[i].size() <= q || cur.ax[i][q] != g.acting[q]) return REDIST_EINTERNAL;
                cur.ax[i].erase(cur.ax[i].begin(), cur.ax[i].begin() + g.acting.size());
                g.post = cur;
                g.local_after = localtype_of(p, cur);
                steps.push_back(g);
            }
            end = cur;
        }

        height = p.local_src;
        cost = 0;
        for (Step &s : steps) {
            i64 before = product(s.local_before), after = product(s.local_after);
            s.localsize_after = after;
            switch (s.kind) {
            case REDIST_STEP_DYNSLICE: s.cost = 0; break;
            case REDIST_STEP_ALLGATHER: s.cost = after; break;
            default: s.cost = before; break;   // alltoall, allpermute
            }
            cost += s.cost;
            height = std::max(height, after);
        }
        if (!same_assignment(p, end, target)) return REDIST_EINTERNAL;
        if (height > std::max(p.local_src, p.local_dst)) return REDIST_EINTERNAL;
        return REDIST_OK;
    };
    redist_status rc = finish(steps, end, p.cost, p.height);
    if (rc != REDIST_OK) return rc;

    // 6. optionally count the permutation: try the sequences whose own cost lies below the total
    //    of the plan found so far, and keep the cheapest total (then the fewest steps)
    if (p.flags & REDIST_COST_PERMUTE) {
        std::vector<std::vector<WeakStep>> near;
        const i64 lat = S.lat;
        i64 best_total = p.cost + lat * i64(steps.size());       // every collective of the plan pays the latency
        S.near(best_total, int(steps.size()) + 3, 256, near);
        for (const auto &cand : near) {
            i64 weak = 0;
            std::vector<Step> st;
            ConcreteState e;
            if (!L.lower(cand, st, e)) continue;
            for (const Step &s : st)
                weak += lat + (s.kind == REDIST_STEP_DYNSLICE    ? 0
                               : s.kind == REDIST_STEP_ALLGATHER ? product(s.local_after)
                                                                 : product(s.local_before));
            if (weak >= best_total) continue;
            i64 cost = 0, height = 0;
            if (finish(st, e, cost, height) != REDIST_OK) continue;
            const i64 total = cost + lat * i64(st.size());
            if (total < best_total || (total == best_total && st.size() < steps.size())) {
                steps = st;
                p.cost = cost;
                p.height = height;
                best_total = total;
            }
        }
    }
    p.steps = steps;
    return REDIST_OK;
}

}  // namespace redist
