// Host-side schedule compiler: integers only.
//
// From the raw schedule (who is active when; which packets are lost or late) it derives what
// Algorithm 1 calls tau_v / tau_rho -- per activation and in-edge, the largest stamp among the
// packets usable by then -- which is the same information as the delays d_v, d_rho that
// Algorithm 2 picks in step S.0.  Every packet payload that some later activation reads is a
// "version"; the compiler computes each version's lifetime and gives it a row in a pool, so
// that the kernels find a delayed payload by row id and a stale payload survives the sender's
// later overwrites without any copy.
#include <algorithm>
#include <climits>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <atomic>
#include <thread>

#include "rfast_internal.h"

namespace rfast {

static int fail(std::string& err, int code, const char* fmt, long long a = 0, long long b = 0,
                long long c = 0) {
    char buf[256];
    std::snprintf(buf, sizeof buf, fmt, a, b, c);
    err = buf;
    return code;
}

int build_host_graph(const rfast_graph& g, int n, bool row_stochastic, HostGraph& H,
                     std::string& err) {
    if (n <= 0 || g.n_edges < 0 || !g.rowptr || !g.diag || (g.n_edges > 0 && (!g.col || !g.w)))
        return fail(err, RFAST_EINVAL, "graph: null array or bad size");
    H.n = n;
    H.E = g.n_edges;
    H.rowptr.assign(g.rowptr, g.rowptr + n + 1);
    if (H.rowptr[0] != 0 || H.rowptr[n] != H.E)
        return fail(err, RFAST_EGRAPH, "graph: rowptr must run from 0 to n_edges");
    H.col.assign(g.col, g.col + H.E);
    H.w.assign(g.w, g.w + H.E);
    H.diag.assign(g.diag, g.diag + n);
    H.recv.resize(H.E);
    for (int i = 0; i < n; ++i) {
        if (H.rowptr[i + 1] < H.rowptr[i])
            return fail(err, RFAST_EGRAPH, "graph: rowptr decreases at node %lld", i);
        if (!(H.diag[i] > 0.f))
            return fail(err, RFAST_EGRAPH, "Assumption 1: diagonal entry of node %lld not positive", i);
        for (int e = H.rowptr[i]; e < H.rowptr[i + 1]; ++e) {
            int j = H.col[e];
            if (j < 0 || j >= n || j == i)
                return fail(err, RFAST_EGRAPH, "graph: bad sender %lld in row %lld", j, i);
            if (e > H.rowptr[i] && H.col[e - 1] >= j)
                return fail(err, RFAST_EGRAPH, "graph: senders of row %lld not strictly ascending", i);
            if (!(H.w[e] > 0.f))
                return fail(err, RFAST_EGRAPH, "Assumption 1: weight of edge %lld not positive", e);
            H.recv[e] = i;
        }
    }
    // Assumption 1 ii): W 1 = 1 (rows), 1^T A = 1^T (columns)
    std::vector<double> sum(n);
    for (int i = 0; i < n; ++i) sum[i] = H.diag[i];
    for (int e = 0; e < H.E; ++e) sum[row_stochastic ? H.recv[e] : H.col[e]] += H.w[e];
    for (int i = 0; i < n; ++i)
        if (std::fabs(sum[i] - 1.0) > 1e-5)
            return fail(err, RFAST_EGRAPH,
                        row_stochastic ? "Assumption 1: row %lld of W does not sum to 1"
                                       : "Assumption 1: column %lld of A does not sum to 1", i);
    // sender-side lists, receivers ascending
    H.optr.assign(n + 1, 0);
    for (int e = 0; e < H.E; ++e) H.optr[H.col[e] + 1]++;
    for (int i = 0; i < n; ++i) H.optr[i + 1] += H.optr[i];
    H.oeid.resize(H.E);
    H.opos.resize(H.E);
    std::vector<int> fill(H.optr.begin(), H.optr.end() - 1);
    for (int e = 0; e < H.E; ++e) {           // edge ids ascend with the receiver
        int j = H.col[e];
        H.opos[e] = fill[j] - H.optr[j];
        H.oeid[fill[j]++] = e;
    }
    return RFAST_OK;
}

// Assumption 2: the root reaches every node along G(W) and along G(A^T).
int check_roots(const HostGraph& R, const HostGraph& C, int root, std::string& err) {
    const int n = R.n;
    if (root < 0 || root >= n) return fail(err, RFAST_EINVAL, "root %lld out of range", root);
    std::vector<char> seen(n, 0);
    std::vector<int> todo;
    auto bfs = [&](bool along_W) {
        std::fill(seen.begin(), seen.end(), 0);
        todo.assign(1, root);
        seen[root] = 1;
        int cnt = 1;
        while (!todo.empty()) {
            int u = todo.back();
            todo.pop_back();
            if (along_W) {                       // u sends to the receivers of its out-edges
                for (int k = R.optr[u]; k < R.optr[u + 1]; ++k) {
                    int v = R.recv[R.oeid[k]];
                    if (!seen[v]) { seen[v] = 1; ++cnt; todo.push_back(v); }
                }
            } else {                             // G(A^T): u -> j whenever A_uj > 0
                for (int e = C.rowptr[u]; e < C.rowptr[u + 1]; ++e) {
                    int v = C.col[e];
                    if (!seen[v]) { seen[v] = 1; ++cnt; todo.push_back(v); }
                }
            }
        }
        return cnt;
    };
    if (bfs(true) != n)
        return fail(err, RFAST_EGRAPH, "Assumption 2: node %lld is not a root of a spanning tree of G(W)", root);
    if (bfs(false) != n)
        return fail(err, RFAST_EGRAPH, "Assumption 2: node %lld is not a root of a spanning tree of G(A^T)", root);
    return RFAST_OK;
}

namespace {
struct Pend { int arrival, stamp; };

// Packets in flight on one edge.  A handful at most in practice (bounded by the largest delay and
// by how long the receiver stays idle), so they live inline; a longer queue spills to the heap.
struct PendQ {
    static constexpr int kInline = 14;
    Pend a[kInline];
    int n = 0;
    std::vector<Pend>* more = nullptr;
    ~PendQ() { delete more; }
    void push(Pend p) {
        if (more) { more->push_back(p); return; }
        if (n < kInline) { a[n++] = p; return; }
        more = new std::vector<Pend>(a, a + n);
        more->push_back(p);
    }
};

// Largest usable stamp on one edge at round r; drops what has arrived from the pending list.
inline int deliver(PendQ& q, int r, int tau) {
    if (q.more) {
        std::vector<Pend>& v = *q.more;
        size_t keep = 0;
        for (size_t k = 0; k < v.size(); ++k) {
            if (v[k].arrival <= r) tau = std::max(tau, v[k].stamp);
            else v[keep++] = v[k];
        }
        v.resize(keep);
        return tau;
    }
    int keep = 0;
    for (int k = 0; k < q.n; ++k) {
        if (q.a[k].arrival <= r) tau = std::max(tau, q.a[k].stamp);
        else q.a[keep++] = q.a[k];
    }
    q.n = keep;
    return tau;
}
}  // namespace

int compile_schedule(const HostGraph& R, const HostGraph& C, const rfast_schedule* s, int batch,
                     int rows, const ModelTraffic& mt, bool buckets, Compiled& out, std::string& err,
                     const std::vector<int>* holds) {
    const int n = R.n;
    if (!s || s->K < 0 || !s->act_ptr) return fail(err, RFAST_ESCHED, "schedule: null or K < 0");
    const int K = s->K;
    if (holds && !holds->empty()) {
        if (buckets) return fail(err, RFAST_ESCHED, "schedule: rounds can be appended to running sums only, not to mass buckets");
        for (size_t k = 0; k < holds->size(); ++k)
            if ((*holds)[k] < 0 || (*holds)[k] > K || (k && (*holds)[k] <= (*holds)[k - 1]))
                return fail(err, RFAST_ESCHED, "schedule: hold rounds must ascend inside 0 .. K");
    }
    if (s->act_ptr[0] != 0) return fail(err, RFAST_ESCHED, "schedule: act_ptr[0] != 0");
    for (int r = 0; r < K; ++r)
        if (s->act_ptr[r + 1] < s->act_ptr[r])
            return fail(err, RFAST_ESCHED, "schedule: act_ptr decreases at round %lld", r);
    const int64_t nE = s->act_ptr[K];
    if (nE > 0 && !s->act_node) return fail(err, RFAST_ESCHED, "schedule: act_node is null");
    Compiled c;
    c.K = K;
    c.n_events = nE;
    c.buckets = buckets;
    c.act_ptr.assign(s->act_ptr, s->act_ptr + K + 1);
    c.act_node.assign(s->act_node, s->act_node + nE);
    c.in_r_off.assign(nE + 1, 0);
    c.in_c_off.assign(nE + 1, 0);
    c.out_r_off.assign(nE + 1, 0);
    c.out_c_off.assign(nE + 1, 0);
    for (int r = 0; r < K; ++r)
        for (int ev = c.act_ptr[r]; ev < c.act_ptr[r + 1]; ++ev) {
            int i = c.act_node[ev];
            if (i < 0 || i >= n) return fail(err, RFAST_ESCHED, "schedule: node id %lld out of range (event %lld)", i, ev);
            if (ev > c.act_ptr[r] && c.act_node[ev - 1] >= i)
                return fail(err, RFAST_ESCHED, "schedule: nodes of round %lld not strictly ascending", r);
            c.in_r_off[ev + 1] = c.in_r_off[ev] + R.indeg(i);
            c.in_c_off[ev + 1] = c.in_c_off[ev] + C.indeg(i);
            c.out_r_off[ev + 1] = c.out_r_off[ev] + R.outdeg(i);
            c.out_c_off[ev + 1] = c.out_c_off[ev] + C.outdeg(i);
        }
    if (s->n_send_r != c.out_r_off[nE] || s->n_send_c != c.out_c_off[nE])
        return fail(err, RFAST_ESCHED, "schedule: send code counts (%lld, %lld) do not match the out-degrees",
                    s->n_send_r, s->n_send_c);
    if ((s->n_send_r > 0 && !s->send_r) || (s->n_send_c > 0 && !s->send_c))
        return fail(err, RFAST_ESCHED, "schedule: send codes are null");
    for (int64_t k = 0; k < s->n_send_r; ++k)
        if (s->send_r[k] < -1) return fail(err, RFAST_ESCHED, "schedule: send_r code below -1 at %lld", k);
    for (int64_t k = 0; k < s->n_send_c; ++k)
        if (s->send_c[k] < -1) return fail(err, RFAST_ESCHED, "schedule: send_c code below -1 at %lld", k);
    if (batch > 0) {
        if (s->n_batch_idx != (int64_t)(n + nE) * batch || !s->batch_idx)
            return fail(err, RFAST_ESCHED, "schedule: batch_idx must hold (n + events) * B = %lld entries",
                        (long long)(n + nE) * batch);
        for (int64_t k = 0; k < s->n_batch_idx; ++k)
            if (s->batch_idx[k] < 0 || s->batch_idx[k] >= rows)
                return fail(err, RFAST_ESCHED, "schedule: batch index out of the shard at %lld", k);
    }

    // ---- pass 1: consumed stamps, version lifetimes -----------------------------------------
    // What an edge delivers depends on that edge alone: the rounds in which its sender sent (with
    // which delay code) and the rounds in which its receiver was active.  So the replay runs edge
    // by edge -- a packet sent in round r with delay d is usable from round r + 1 + d, a receiver
    // active in round r takes the largest stamp usable by then -- and long schedules spread the
    // edges over several threads.  Every edge writes its own entries only.
    const int INF = INT_MAX;
    std::vector<int> tau_v(R.E, 0), tau_rho(C.E, 0), t(n, 0);
    c.ev_of.assign(n, {});
    {
        std::vector<int> cnt(n, 0);
        for (int64_t ev = 0; ev < nE; ++ev) cnt[c.act_node[ev]]++;
        for (int i = 0; i < n; ++i) c.ev_of[i].reserve(cnt[i]);
    }
    std::vector<std::vector<int>>& ev_of = c.ev_of;    // node -> event id of stamp s at [s-1]
    std::vector<int> ev_round(nE);
    c.used_tau_v.assign(c.in_r_off[nE], 0);
    c.used_tau_rho.assign(c.in_c_off[nE], 0);
    c.prev_tau_rho.assign(c.in_c_off[nE], 0);
    c.v_write.assign(nE, 0);
    c.v_last.assign(nE, 0);
    std::vector<char> v_sent(nE, 0);
    const int64_t nRho = c.out_c_off[nE];
    c.rho_write.assign(nRho, 0);
    std::vector<int> rho_last_sender(nRho, 0), rho_last_recv(nRho, -1);
    std::vector<int> v_last_edge(c.out_r_off[nE], -1);     // per (event, G_R out-edge): last round its v is read
    if (buckets) c.rho_leader.assign(nRho, -1);
    for (int r = 0; r < K; ++r)
        for (int ev = c.act_ptr[r]; ev < c.act_ptr[r + 1]; ++ev) {
            const int i = c.act_node[ev];
            ev_round[ev] = r;
            ev_of[i].push_back(ev);
            c.v_write[ev] = r;
            for (int k = 0; k < R.outdeg(i); ++k) v_sent[ev] |= s->send_r[c.out_r_off[ev] + k] >= 0;
            for (int k = 0; k < C.outdeg(i); ++k) { c.rho_write[c.out_c_off[ev] + k] = r; rho_last_sender[c.out_c_off[ev] + k] = r; }
        }
    for (int i = 0; i < n; ++i) {
        t[i] = (int)ev_of[i].size();
        if (!buckets)                                     // S2c of the next activation reads the sender's current running sums
            for (size_t q = 0; q + 1 < ev_of[i].size(); ++q) {
                const int64_t base = c.out_c_off[ev_of[i][q]];
                for (int k = 0; k < C.outdeg(i); ++k) rho_last_sender[base + k] = ev_round[ev_of[i][q + 1]];
            }
    }
    // A hold at round b: whatever an activation in round b or later may still read stays in its
    // row through round b -- per edge the version its receiver holds and every packet still on
    // its way or waiting, and every sender's latest running sums.  The rows of the rounds before
    // b then do not depend on what follows b: rounds can be appended without moving any of them.
    static const std::vector<int> no_holds;
    const std::vector<int>& H = holds ? *holds : no_holds;
    auto for_pending = [](const PendQ& q, auto&& f) {
        if (q.more) { for (const Pend& pk : *q.more) f(pk); }
        else for (int k = 0; k < q.n; ++k) f(q.a[k]);
    };
    auto edge_r = [&](int e) {
        const std::vector<int>& S = ev_of[R.col[e]];
        const std::vector<int>& A = ev_of[R.recv[e]];
        const int kin = e - R.rowptr[R.recv[e]], kout = R.opos[e];
        PendQ q;
        int tau = 0;
        size_t ps = 0, h = 0;
        auto read_in = [&](int stamp, int r) { int& l = v_last_edge[c.out_r_off[S[stamp - 1]] + kout]; l = std::max(l, r); };
        auto admit = [&](int before) {                       // the packets sent in rounds < before
            for (; ps < S.size() && ev_round[S[ps]] < before; ++ps) {
                const int d = s->send_r[c.out_r_off[S[ps]] + kout];
                if (d >= 0) q.push({ev_round[S[ps]] + 1 + d, (int)ps + 1});
            }
        };
        auto hold = [&](int b) {
            admit(b);
            if (tau >= 1) read_in(tau, b);
            for_pending(q, [&](const Pend& pk) { if (pk.stamp > tau) read_in(pk.stamp, b); });
        };
        for (int ev : A) {
            const int r = ev_round[ev];
            for (; h < H.size() && H[h] <= r; ++h) hold(H[h]);
            admit(r);
            tau = deliver(q, r, tau);
            c.used_tau_v[c.in_r_off[ev] + kin] = tau;
            if (tau >= 1) read_in(tau, r);
        }
        for (; h < H.size(); ++h) hold(H[h]);
        tau_v[e] = tau;
    };
    auto edge_c = [&](int e) {
        const std::vector<int>& S = ev_of[C.col[e]];
        const std::vector<int>& A = ev_of[C.recv[e]];
        const int kin = e - C.rowptr[C.recv[e]], kout = C.opos[e];
        PendQ q;
        int tau = 0;
        size_t ps = 0, h = 0;
        auto vid_of = [&](int stamp) { return c.out_c_off[S[stamp - 1]] + kout; };
        auto read_in = [&](int stamp, int r) { int& l = rho_last_recv[vid_of(stamp)]; l = std::max(l, r); };
        auto admit = [&](int before) {
            for (; ps < S.size() && ev_round[S[ps]] < before; ++ps) {
                const int d = s->send_c[c.out_c_off[S[ps]] + kout];
                if (d >= 0) q.push({ev_round[S[ps]] + 1 + d, (int)ps + 1});
            }
        };
        auto hold = [&](int b) {
            admit(b);
            if (tau >= 1) read_in(tau, b);
            for_pending(q, [&](const Pend& pk) { if (pk.stamp > tau) read_in(pk.stamp, b); });
        };
        for (int ev : A) {
            const int r = ev_round[ev];
            for (; h < H.size() && H[h] <= r; ++h) hold(H[h]);
            admit(r);
            const int prev = tau;
            tau = deliver(q, r, prev);
            c.used_tau_rho[c.in_c_off[ev] + kin] = tau;
            c.prev_tau_rho[c.in_c_off[ev] + kin] = prev;
            if (tau > prev && buckets) {                   // news: the contributions of stamps prev+1 .. tau, one row
                const int64_t lead = vid_of(prev + 1);
                for (int st = prev + 1; st <= tau; ++st) c.rho_leader[vid_of(st)] = lead;
                rho_last_recv[lead] = r;
            } else if (tau > prev) {                       // news: rho[tau] - rho[prev] is read
                read_in(tau, r);
                if (prev >= 1) read_in(prev, r);
            }
        }
        for (; h < H.size(); ++h) hold(H[h]);
        tau_rho[e] = tau;
    };
    {
        int nthreads = 1;
        if (nE >= 50000) nthreads = (int)std::min<unsigned>(8u, std::max(1u, std::thread::hardware_concurrency()));
        if (const char* cap = std::getenv("RFAST_COMPILE_THREADS")) nthreads = std::max(1, std::min(nthreads, std::atoi(cap)));
        std::atomic<int> next{0};
        auto work = [&]() {
            for (int e; (e = next.fetch_add(1)) < R.E + C.E;) {
                if (e < R.E) edge_r(e); else edge_c(e - R.E);
            }
        };
        if (nthreads == 1) work();
        else {
            std::vector<std::thread> pool;
            for (int th = 0; th < nthreads; ++th) pool.emplace_back(work);
            for (auto& t_ : pool) t_.join();
        }
    }
    for (int64_t ev = 0; ev < nE; ++ev) {
        int last = c.v_write[ev];
        for (int64_t q = c.out_r_off[ev]; q < c.out_r_off[ev + 1]; ++q) last = std::max(last, v_last_edge[q]);
        c.v_last[ev] = last;
    }
    for (int b : H)                                        // every sender's latest running sums as of round b
        for (int i = 0; i < n; ++i) {
            const auto& evs = ev_of[i];
            const size_t tb = std::lower_bound(evs.begin(), evs.end(), b, [&](int ev, int rb) { return ev_round[ev] < rb; }) - evs.begin();
            if (tb >= 1) {
                const int64_t base = c.out_c_off[evs[tb - 1]];
                for (int k = 0; k < C.outdeg(i); ++k) rho_last_sender[base + k] = std::max(rho_last_sender[base + k], b);
            }
        }
    c.tau_v_end = tau_v;
    c.tau_rho_end = tau_rho;
    c.t_end = t;
    if (buckets) {
        // contributions nobody consumes inside the schedule: one last bucket per edge, kept
        for (int e = 0; e < C.E; ++e) {
            const int j = C.col[e];
            if (t[j] <= tau_rho[e]) continue;
            const int64_t lead = c.out_c_off[ev_of[j][tau_rho[e]]] + C.opos[e];
            for (int st = tau_rho[e] + 1; st <= t[j]; ++st) c.rho_leader[c.out_c_off[ev_of[j][st - 1]] + C.opos[e]] = lead;
            rho_last_recv[lead] = INF;
        }
        c.rho_last.resize(nRho);
        for (int64_t v = 0; v < nRho; ++v) c.rho_last[v] = rho_last_recv[c.rho_leader[v]];
    } else {
    // what is current at the end of the schedule stays readable: each sender's latest running
    // sums and each receiver's buffered version
    for (int i = 0; i < n; ++i)
        if (t[i] >= 1) {
            int64_t base = c.out_c_off[ev_of[i][t[i] - 1]];
            for (int k = 0; k < C.outdeg(i); ++k) rho_last_sender[base + k] = INF;
        }
    for (int e = 0; e < C.E; ++e)
        if (tau_rho[e] >= 1)
            rho_last_recv[c.out_c_off[ev_of[C.col[e]][tau_rho[e] - 1]] + C.opos[e]] = INF;
    c.rho_last.resize(nRho);
    for (int64_t v = 0; v < nRho; ++v) c.rho_last[v] = std::max(rho_last_sender[v], rho_last_recv[v]);
    }

    // ---- pass 2: rows.  A row is free again in the round after its version's last read -------
    c.v_slot.assign(nE, -1);
    c.rho_slot.assign(nRho, -1);
    std::vector<std::vector<int64_t>> rel_v(K + 1), rel_c(K + 1);
    std::vector<int> free_v, free_c;
    std::vector<char> moved(nRho, 0);                  // row handed on to the next version in place
    std::vector<int> stamp_of(nE, 0);
    {
        std::vector<int> tt(n, 0);
        for (int64_t ev = 0; ev < nE; ++ev) stamp_of[ev] = ++tt[c.act_node[ev]];
    }
    for (int r = 0; r < K; ++r) {
        for (int64_t id : rel_v[r]) free_v.push_back(c.v_slot[id]);
        for (int64_t id : rel_c[r]) if (!moved[id]) free_c.push_back(c.rho_slot[id]);
        for (int ev = c.act_ptr[r]; ev < c.act_ptr[r + 1]; ++ev) {
            const int i = c.act_node[ev];
            if (v_sent[ev]) {
                int slot;
                if (!free_v.empty()) { slot = free_v.back(); free_v.pop_back(); }
                else slot = c.n_v_slots++;
                c.v_slot[ev] = slot;
                if (c.v_last[ev] + 1 < K) rel_v[c.v_last[ev] + 1].push_back(ev);
            }
            for (int k = 0; k < C.outdeg(i); ++k) {
                int64_t vid = c.out_c_off[ev] + k;
                int slot = -1;
                if (buckets) {                         // the first contribution of a bucket takes a row, the others share it
                    const int64_t lead = c.rho_leader[vid];
                    if (lead != vid) { c.rho_slot[vid] = c.rho_slot[lead]; continue; }
                    if (!free_c.empty()) { slot = free_c.back(); free_c.pop_back(); }
                    else slot = c.n_rho_slots++;
                    c.rho_slot[vid] = slot;
                    if (c.rho_last[vid] != INF && c.rho_last[vid] + 1 < K) rel_c[c.rho_last[vid] + 1].push_back(vid);
                    continue;
                }
                if (stamp_of[ev] >= 2) {
                    // in place: the previous version is read for the last time here, by this
                    // very update, and no receiver reads it in this round or later
                    int64_t cur = c.out_c_off[ev_of[i][stamp_of[ev] - 2]] + k;
                    if (c.rho_last[cur] == r && rho_last_recv[cur] < r) {
                        slot = c.rho_slot[cur];
                        moved[cur] = 1;
                    }
                }
                if (slot < 0) {
                    if (!free_c.empty()) { slot = free_c.back(); free_c.pop_back(); }
                    else slot = c.n_rho_slots++;
                }
                c.rho_slot[vid] = slot;
                if (c.rho_last[vid] != INF && c.rho_last[vid] + 1 < K)
                    rel_c[c.rho_last[vid] + 1].push_back(vid);
            }
        }
    }

    // ---- pass 3: device descriptors and the method's traffic ---------------------------------
    // Rounds are independent of one another here once every list's starting offset is known, so
    // long schedules are filled in by several threads, each on a contiguous span of rounds.
    c.ev.resize(nE);
    c.round_streams.assign(K + 1, 0);
    c.round_streams_method.assign(K + 1, 0);
    std::vector<int64_t> mix_at(K + 1, 0), news_at(K + 1, 0);          // list offsets at the start of each round
    for (int r = 0; r < K; ++r) {
        int64_t nm = 0, nn = 0;
        for (int64_t q = c.in_r_off[c.act_ptr[r]]; q < c.in_r_off[c.act_ptr[r + 1]]; ++q) nm += c.used_tau_v[q] >= 1;
        for (int64_t q = c.in_c_off[c.act_ptr[r]]; q < c.in_c_off[c.act_ptr[r + 1]]; ++q) nn += c.used_tau_rho[q] > c.prev_tau_rho[q];
        mix_at[r + 1] = mix_at[r] + nm;
        news_at[r + 1] = news_at[r] + nn;
    }
    c.mix_slot.resize(mix_at[K]);  c.mix_w.resize(mix_at[K]);
    c.news_new.resize(news_at[K]);  c.news_prev.resize(news_at[K]);  c.news_edge.resize(news_at[K]);
    c.out_cur.resize(nRho);  c.out_new.resize(nRho);  c.out_a.resize(nRho);  c.out_edge.resize(nRho);
    std::vector<int64_t> round_s(K, 0), round_m(K, 0);
    auto fill = [&](int r_begin, int r_end, int64_t* bad_event) {
        for (int r = r_begin; r < r_end; ++r) {
            int64_t streams = 0, method = 0, mix_pos = mix_at[r], news_pos = news_at[r];
            for (int ev = c.act_ptr[r]; ev < c.act_ptr[r + 1]; ++ev) {
                const int i = c.act_node[ev];
                EvDesc d{};
                d.node = i;
                d.v_out = c.v_slot[ev];
                d.w_self = R.diag[i];
                d.a_self = C.diag[i];
                d.stamp = stamp_of[ev];
                d.g_par = (stamp_of[ev] - 1) & 1;
                d.sample = (int32_t)(n + ev);
                d.mix_beg = (int32_t)mix_pos;
                for (int e = R.rowptr[i], k = 0; e < R.rowptr[i + 1]; ++e, ++k) {
                    int tau = c.used_tau_v[c.in_r_off[ev] + k];
                    if (tau < 1) continue;                 // stamp 0 is the zero vector: nothing to read
                    int slot = c.v_slot[ev_of[R.col[e]][tau - 1]];
                    if (slot < 0 && *bad_event < 0) *bad_event = ev;
                    c.mix_slot[mix_pos] = slot;
                    c.mix_w[mix_pos++] = R.w[e];
                }
                d.mix_cnt = (int32_t)mix_pos - d.mix_beg;
                d.news_beg = (int32_t)news_pos;
                int news_streams = 0;
                for (int e = C.rowptr[i], k = 0; e < C.rowptr[i + 1]; ++e, ++k) {
                    int tau = c.used_tau_rho[c.in_c_off[ev] + k];
                    int prev = c.prev_tau_rho[c.in_c_off[ev] + k];
                    if (tau <= prev) continue;             // nothing newer: rho[tau] - rho~ = 0
                    const auto& evs = ev_of[C.col[e]];
                    c.news_new[news_pos] = c.rho_slot[c.out_c_off[evs[tau - 1]] + C.opos[e]];
                    const bool sub = !buckets && prev >= 1;   // a bucket holds the difference itself
                    c.news_prev[news_pos] = sub ? c.rho_slot[c.out_c_off[evs[prev - 1]] + C.opos[e]] : -1;
                    c.news_edge[news_pos++] = e;
                    news_streams += 1 + sub;
                }
                d.news_cnt = (int32_t)news_pos - d.news_beg;
                d.out_beg = (int32_t)c.out_c_off[ev];
                int out_streams = 0;
                for (int k = 0; k < C.outdeg(i); ++k) {
                    const int64_t vid = c.out_c_off[ev] + k;
                    int e = C.oeid[C.optr[i] + k];
                    int cur = -1;
                    if (buckets) {                         // add to the bucket unless this is its first contribution
                        if (c.rho_leader[vid] != vid) cur = c.rho_slot[vid];
                    } else if (stamp_of[ev] >= 2) cur = c.rho_slot[c.out_c_off[ev_of[i][stamp_of[ev] - 2]] + k];
                    c.out_cur[vid] = cur;
                    c.out_new[vid] = c.rho_slot[vid];
                    c.out_a[vid] = C.w[e];
                    c.out_edge[vid] = e;
                    out_streams += 1 + (cur >= 0);
                }
                d.out_cnt = C.outdeg(i);
                c.ev[ev] = d;
                // fp32 streams per coordinate: S1/S2a read x, z, the neighbours' v, write v (if a
                // packet leaves) and x; S2b/S2c read the news, write z and the running sums
                const int64_t base = 2 + d.mix_cnt + (d.v_out >= 0) + 1 + news_streams + 1 + out_streams;
                streams += base + (mt.elementwise ? mt.data_streams : mt.grad_track_streams);
                // what the method itself must move: x and z read once, the gradient moved once
                // (remembered one read, new one written), no stream that exists only because the
                // step is split over several kernels or because of the tracker's arithmetic
                method += base + mt.method_streams;
            }
            round_s[r] = streams;
            round_m[r] = method;
        }
    };
    {
        int nthreads = 1;
        if (nE >= 50000) nthreads = (int)std::min<unsigned>(8u, std::max(1u, std::thread::hardware_concurrency()));
        if (const char* cap = std::getenv("RFAST_COMPILE_THREADS")) nthreads = std::max(1, std::min(nthreads, std::atoi(cap)));
        std::vector<int64_t> bad(nthreads, -1);
        if (nthreads == 1) {
            fill(0, K, &bad[0]);
        } else {
            std::vector<std::thread> pool;
            int r0 = 0;
            for (int th = 0; th < nthreads; ++th) {             // spans of about equally many events
                const int64_t target = nE * (th + 1) / nthreads;
                int r1 = th + 1 == nthreads ? K : r0;
                while (th + 1 < nthreads && r1 < K && c.act_ptr[r1] < target) ++r1;
                pool.emplace_back(fill, r0, r1, &bad[th]);
                r0 = r1;
            }
            for (auto& t_ : pool) t_.join();
        }
        for (int64_t bev : bad)
            if (bev >= 0) return fail(err, RFAST_ESCHED, "internal: consumed v version without a row (event %lld)", bev);
    }
    // Every index a kernel will dereference is checked here, on the host, before anything is
    // launched: rows inside their pools, list ranges inside their lists, node ids inside the state.
    {
        const int64_t n_mix = (int64_t)c.mix_slot.size(), n_news = (int64_t)c.news_new.size();
        for (int64_t ev = 0; ev < nE; ++ev) {
            const EvDesc& d = c.ev[ev];
            bool good = d.node >= 0 && d.node < n && d.v_out >= -1 && d.v_out < c.n_v_slots &&
                        d.mix_beg >= 0 && d.mix_cnt >= 0 && (int64_t)d.mix_beg + d.mix_cnt <= n_mix &&
                        d.news_beg >= 0 && d.news_cnt >= 0 && (int64_t)d.news_beg + d.news_cnt <= n_news &&
                        d.out_beg >= 0 && d.out_cnt >= 0 && (int64_t)d.out_beg + d.out_cnt <= nRho &&
                        (d.g_par == 0 || d.g_par == 1) && d.sample >= n && (int64_t)d.sample < n + nE;
            for (int m = 0; good && m < d.mix_cnt; ++m)
                good = c.mix_slot[d.mix_beg + m] >= 0 && c.mix_slot[d.mix_beg + m] < c.n_v_slots;
            for (int m = 0; good && m < d.news_cnt; ++m)
                good = c.news_new[d.news_beg + m] >= 0 && c.news_new[d.news_beg + m] < c.n_rho_slots &&
                       c.news_prev[d.news_beg + m] >= -1 && c.news_prev[d.news_beg + m] < c.n_rho_slots;
            for (int m = 0; good && m < d.out_cnt; ++m)
                good = c.out_new[d.out_beg + m] >= 0 && c.out_new[d.out_beg + m] < c.n_rho_slots &&
                       c.out_cur[d.out_beg + m] >= -1 && c.out_cur[d.out_beg + m] < c.n_rho_slots;
            if (!good) return fail(err, RFAST_ESCHED, "internal: descriptor of event %lld points outside its pools or lists", ev);
        }
    }
    for (int r = 0; r < K; ++r) {
        c.round_streams[r + 1] = c.round_streams[r] + round_s[r];
        c.round_streams_method[r + 1] = c.round_streams_method[r] + round_m[r];
    }
    out = std::move(c);
    return RFAST_OK;
}

}  // namespace rfast
