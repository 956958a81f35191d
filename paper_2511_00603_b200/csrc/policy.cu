// Host-side policies around the serving step (no device code): the request handler's offloading rule
// (paper Section 3.2, Eq. 1), an event-driven simulator with lookup-table compute latencies (Section 5.2)
// that evaluates the placement objective (Eq. 2) under the handler's decision list, and the state-aware
// submodular placement (Algorithm 1 over Algorithm 2).  The compute-time tables are what the allocator's
// offline profiler measures on this library's kernels (Section 4.1).
#include <algorithm>
#include <cmath>
#include <functional>
#include <map>
#include <queue>
#include <tuple>
#include <utility>
#include <vector>

#include "../../include/epara.h"

namespace {

typedef std::pair<int, int> Placement;   // (service, server); server == n_servers is the hypothetical server

double lookup_ms(const epara_service& s, int batch) {
  int k = 0;
  while ((1 << k) < batch && k + 1 < EPARA_PROFILE_POINTS) ++k;
  return s.c_ms[k];
}

struct Usage {
  std::vector<std::vector<std::pair<double, double>>> gpu;   // [server][gpu] = (compute used, VRAM used)
  explicit Usage(const epara_cluster& c) {
    gpu.resize(c.n_servers);
    for (int n = 0; n < c.n_servers; ++n) gpu[n].assign(c.gpus[n], std::make_pair(0.0, 0.0));
  }
};

// First fit in (server, gpu) order: the first n_gpus GPUs with the service's compute share and VRAM free, all on
// server n, or on any servers when n is the hypothetical server.
bool try_place(const epara_cluster& c, const epara_service* sv, Usage& u, int l, int n) {
  const epara_service& s = sv[l];
  std::vector<std::pair<int, int>> got;
  const int lo = (n == c.n_servers) ? 0 : n, hi = (n == c.n_servers) ? c.n_servers : n + 1;
  for (int x = lo; x < hi; ++x)
    for (int y = 0; y < c.gpus[x]; ++y) {
      if (u.gpu[x][y].first + s.a <= 1.0 + 1e-12 && u.gpu[x][y].second + s.b <= c.vram + 1e-12) {
        got.push_back(std::make_pair(x, y));
        if ((int)got.size() == s.n_gpus) {
          for (auto& g : got) { u.gpu[g.first][g.second].first += s.a; u.gpu[g.first][g.second].second += s.b; }
          return true;
        }
      }
    }
  return false;
}

bool feasible(const epara_cluster& c, const epara_service* sv, const std::vector<Placement>& th) {
  Usage u(c);
  for (const Placement& p : th)
    if (!try_place(c, sv, u, p.first, p.second)) return false;
  return true;
}

void offload_prob(int n, const double* p_hat, const double* p_act, const double* queued_ms, const double* t_sync_ms,
                  double slo_ms, double* prob) {
  double sum = 0.0;
  for (int m = 0; m < n; ++m) {
    const bool ok = queued_ms[m] <= t_sync_ms[m] + slo_ms;
    prob[m] = ok ? std::max(0.0, p_hat[m] - p_act[m]) : 0.0;
    sum += prob[m];
  }
  for (int m = 0; m < n; ++m) prob[m] = sum > 0 ? prob[m] / sum : 0.0;
}

int pick(const std::vector<double>& prob, double u) {
  double acc = 0.0;
  int last = -1;
  for (int m = 0; m < (int)prob.size(); ++m) {
    if (prob[m] <= 0) continue;
    acc += prob[m];
    last = m;
    if (u < acc) return m;
  }
  return last;
}

struct Instance {
  int l, n;
  std::vector<int> queue, batch;
  double busy_until = 0.0;
  bool running = false;
  std::vector<double> done_times;
};

struct Item {
  int req, l, count;
  double arrive, deadline, done;
  bool has_done;
  std::vector<int> path;
};

struct Event {
  double t;
  long long seq;
  int kind, a, b;
  bool operator>(const Event& o) const { return t != o.t ? t > o.t : seq > o.seq; }
};

// One replay of the requests under the handler's decision list (Section 3.2): timeout, local, offloading
// exceed, offload by Eq. 1, resource insufficiency.  See epara.h for the model.
void simulate(const epara_cluster& c, const epara_service* sv, const epara_request* rq, int n_req,
              const std::vector<Placement>& placements, int max_offload, epara_sim_result* out) {
  const int N = c.n_servers;
  const double t_sync = c.sync_ms;
  Usage usage(c);
  std::vector<Instance> insts;
  for (const Placement& p : placements)
    if (try_place(c, sv, usage, p.first, p.second)) { Instance it; it.l = p.first; it.n = p.second; insts.push_back(it); }
  std::map<std::pair<int, int>, std::vector<int>> by_server;
  for (int i = 0; i < (int)insts.size(); ++i) by_server[std::make_pair(insts[i].n, insts[i].l)].push_back(i);

  std::vector<Item> items;
  std::priority_queue<Event, std::vector<Event>, std::greater<Event>> events;
  long long seq = 0;
  for (int r = 0; r < n_req; ++r) {
    const epara_service& s = sv[rq[r].service];
    const int nf = s.cat == 1 ? s.frames : 1;
    for (int f = 0; f < nf; ++f) {
      Item it;
      it.req = r; it.l = rq[r].service; it.count = 0; it.has_done = false; it.done = 0.0;
      it.arrive = rq[r].t_ms + (s.cat == 1 ? 1000.0 * f / s.fps : 0.0);
      it.deadline = it.arrive + s.slo_ms;
      it.path.push_back(rq[r].server);
      items.push_back(it);
      events.push(Event{it.arrive, seq++, 0, (int)items.size() - 1, rq[r].server});
    }
  }
  epara_sim_result res;
  res.phi = 0.0;
  res.served = res.timeout = res.offload_exceed = res.insufficient = res.late = res.offloads = 0;
  res.instances = (int)insts.size();

  auto queued_ms = [&](int i, double now, int extra) {
    const Instance& it = insts[i];
    const epara_service& s = sv[it.l];
    const double left = it.running ? std::max(0.0, it.busy_until - now) : 0.0;
    const int q = (int)it.queue.size() + extra;
    const int full = q / s.bs, rest = q % s.bs;
    return left + full * lookup_ms(s, s.bs) + (rest ? lookup_ms(s, rest) : 0.0);
  };
  auto start = [&](int i, double now) {
    Instance& it = insts[i];
    const epara_service& s = sv[it.l];
    std::vector<int> live;
    for (int w : it.queue) {
      if (items[w].deadline < now) ++res.timeout; else live.push_back(w);
    }
    const size_t take = std::min(live.size(), (size_t)s.bs);
    it.batch.assign(live.begin(), live.begin() + take);
    it.queue.assign(live.begin() + take, live.end());
    if (it.batch.empty()) { it.running = false; return; }
    it.running = true;
    it.busy_until = now + lookup_ms(s, (int)it.batch.size());
    events.push(Event{it.busy_until, seq++, 1, i, 0});
  };

  while (!events.empty()) {
    const Event e = events.top();
    events.pop();
    const double now = e.t;
    if (e.kind == 1) {
      Instance& it = insts[e.a];
      for (int w : it.batch) {
        items[w].done = now; items[w].has_done = true;
        it.done_times.push_back(now);
        if (now <= items[w].deadline) ++res.served; else ++res.late;
      }
      it.running = false;
      if (!it.queue.empty()) start(e.a, now);
      continue;
    }
    const int w = e.a, n = e.b;
    Item& item = items[w];
    const epara_service& s = sv[item.l];
    if (item.deadline < now) { ++res.timeout; continue; }                       // 1. timed out
    int best = -1;
    double best_t = INFINITY;
    for (int srv : {n, N}) {                                                    // 2. local, then the hypothetical server
      auto f = by_server.find(std::make_pair(srv, item.l));
      if (f != by_server.end())
        for (int i : f->second) {
          const double t_fin = queued_ms(i, now, 1);
          if (now + t_fin <= item.deadline && t_fin < best_t) { best = i; best_t = t_fin; }
        }
      if (best >= 0) break;
    }
    if (best >= 0) {
      insts[best].queue.push_back(w);
      if (!insts[best].running) start(best, now);
      continue;
    }
    if (item.count >= max_offload) { ++res.offload_exceed; continue; }           // 3. offloading exceed
    std::vector<int> cand;                                                      // 4. Eq. 1
    for (int m = 0; m < N; ++m) {
      if (std::find(item.path.begin(), item.path.end(), m) != item.path.end()) continue;
      auto f = by_server.find(std::make_pair(m, item.l));
      if (f != by_server.end() && !f->second.empty()) cand.push_back(m);
    }
    std::vector<double> p_hat, p_act, q_ms, ts, prob(cand.size());
    for (int m : cand) {
      const std::vector<int>& ids = by_server[std::make_pair(m, item.l)];
      double ph = 0.0;
      for (size_t k = 0; k < ids.size(); ++k) ph += s.bs / lookup_ms(s, s.bs) * 1000.0;
      int done = 0;
      double qmin = INFINITY;
      for (int i : ids) {
        for (double d : insts[i].done_times) done += (now - 2 * t_sync <= d && d <= now - t_sync);
        qmin = std::min(qmin, queued_ms(i, now, 0));
      }
      p_hat.push_back(ph);
      p_act.push_back(t_sync > 0 ? done / t_sync * 1000.0 : 0.0);
      q_ms.push_back(qmin);
      ts.push_back(t_sync);
    }
    offload_prob((int)cand.size(), p_hat.data(), p_act.data(), q_ms.data(), ts.data(), s.slo_ms, prob.data());
    const int k = pick(prob, rq[item.req].u[item.count]);
    if (k < 0) { ++res.insufficient; continue; }
    item.count++;
    item.path.push_back(cand[k]);
    ++res.offloads;
    events.push(Event{now + c.offload_ms, seq++, 0, w, cand[k]});
  }

  // Eq. 2: latency-sensitive requests count 1 when in time; a frequency-sensitive request of F frames counts
  // F x achieved / required frame rate, at most the frames that were in time
  std::vector<std::vector<int>> per_req(n_req);
  for (int w = 0; w < (int)items.size(); ++w) per_req[items[w].req].push_back(w);
  for (int r = 0; r < n_req; ++r) {
    const epara_service& s = sv[rq[r].service];
    const std::vector<int>& its = per_req[r];
    if (its.empty()) continue;
    if (s.cat == 0) {
      const Item& it = items[its[0]];
      res.phi += (it.has_done && it.done <= it.deadline) ? 1.0 : 0.0;
    } else {
      int n_done = 0;
      double last = 0.0;
      for (int w : its)
        if (items[w].has_done && items[w].done <= items[w].deadline) { ++n_done; last = std::max(last, items[w].done); }
      if (n_done > 0) {
        const double span_ms = last - items[its[0]].arrive;
        const double achieved = span_ms > 0 ? n_done / (span_ms / 1000.0) : INFINITY;
        const double capped = std::min(achieved, s.fps * n_done / (double)its.size());
        res.phi += (double)its.size() * std::min(1.0, capped / s.fps);
      }
    }
  }
  *out = res;
}

// Algorithm 2: greedy rounds with a tie set; ">=" keeps stage 1 going, ">" the other stages.
std::vector<Placement> spf(const std::function<double(const std::vector<Placement>&)>& phi,
                           const std::function<bool(const std::vector<Placement>&)>& feas,
                           const std::vector<Placement>& X, const std::vector<Placement>& theta0, bool is_set, bool stage1) {
  std::vector<std::vector<Placement>> thetas(1, theta0);
  std::vector<double> phis(1, phi(theta0));
  int k = 0;
  for (;;) {
    ++k;
    const std::vector<Placement>& prev = thetas[k - 1];
    std::vector<Placement> cands;
    if (is_set) {
      cands = X;
    } else {
      std::vector<Placement> left = prev;
      for (const Placement& d : X) {
        auto f = std::find(left.begin(), left.end(), d);
        if (f != left.end()) left.erase(f); else cands.push_back(d);
      }
    }
    std::vector<Placement> tie;
    double tie_val = 0.0;
    for (const Placement& d : cands) {
      std::vector<Placement> th = prev;
      th.push_back(d);
      if (!feas(th)) continue;
      const double v = phi(th);
      if (tie.empty() || v > tie_val) { tie.assign(1, d); tie_val = v; }
      else if (v == tie_val) tie.push_back(d);
    }
    if (tie.empty()) break;
    std::vector<Placement> next = prev;
    next.push_back(tie[0]);                       // "arbitrary": the first of the tie set in X's order
    thetas.push_back(next);
    phis.push_back(tie_val);
    const bool go_on = stage1 ? phis[k] >= phis[k - 1] : phis[k] > phis[k - 1];
    if (!go_on) break;
  }
  return thetas[k - 1];
}

bool valid_model(const epara_cluster* c, const epara_service* sv, int n_services, const epara_request* rq, int n_req) {
  if (!c || c->n_servers <= 0 || !c->gpus || !sv || n_services <= 0 || n_req < 0 || (n_req > 0 && !rq)) return false;
  for (int n = 0; n < c->n_servers; ++n) if (c->gpus[n] < 0) return false;
  for (int l = 0; l < n_services; ++l) {
    const epara_service& s = sv[l];
    if (s.bs <= 0 || s.n_gpus <= 0 || s.a < 0 || s.b < 0 || (s.cat != 0 && s.cat != 1)) return false;
    if (s.cat == 1 && (s.fps <= 0 || s.frames <= 0)) return false;
    for (int k = 0; k < EPARA_PROFILE_POINTS; ++k) if (!(s.c_ms[k] > 0)) return false;
  }
  for (int r = 0; r < n_req; ++r)
    if (rq[r].service < 0 || rq[r].service >= n_services || rq[r].server < 0 || rq[r].server >= c->n_servers) return false;
  return true;
}

}  // namespace

extern "C" {

int epara_offload_probabilities(int n, const double* p_hat, const double* p_act, const double* queued_ms,
                                const double* t_sync_ms, double slo_ms, double* prob) {
  if (n < 0 || (n > 0 && (!p_hat || !p_act || !queued_ms || !t_sync_ms || !prob))) return EPARA_E_INVALID;
  offload_prob(n, p_hat, p_act, queued_ms, t_sync_ms, slo_ms, prob);
  return EPARA_OK;
}

int epara_simulate(const epara_cluster* c, const epara_service* services, int n_services, const epara_request* requests,
                   int n_requests, const epara_placement* placements, int n_placements, int max_offload,
                   epara_sim_result* out) {
  if (!out || n_placements < 0 || (n_placements > 0 && !placements) || max_offload < 0 ||
      max_offload > EPARA_MAX_OFFLOAD_DRAWS || !valid_model(c, services, n_services, requests, n_requests))
    return EPARA_E_INVALID;
  std::vector<Placement> th;
  for (int i = 0; i < n_placements; ++i) {
    if (placements[i].service < 0 || placements[i].service >= n_services || placements[i].server < 0 ||
        placements[i].server > c->n_servers)
      return EPARA_E_INVALID;
    th.push_back(std::make_pair(placements[i].service, placements[i].server));
  }
  simulate(*c, services, requests, n_requests, th, max_offload, out);
  return EPARA_OK;
}

int epara_place_sssp(const epara_cluster* c, const epara_service* services, int n_services, const epara_request* requests,
                     int n_requests, const epara_placement* priority, int n_priority, int max_offload,
                     epara_placement* out, int out_cap, int* n_out) {
  if (!n_out || out_cap < 0 || (out_cap > 0 && !out) || n_priority < 0 || (n_priority > 0 && !priority) || max_offload < 0 ||
      max_offload > EPARA_MAX_OFFLOAD_DRAWS || !valid_model(c, services, n_services, requests, n_requests))
    return EPARA_E_INVALID;
  const int N = c->n_servers;
  std::function<double(const std::vector<Placement>&)> phi = [&](const std::vector<Placement>& th) {
    epara_sim_result r;
    simulate(*c, services, requests, n_requests, th, max_offload, &r);
    return r.phi;
  };
  std::function<bool(const std::vector<Placement>&)> feas = [&](const std::vector<Placement>& th) {
    return feasible(*c, services, th);
  };
  std::vector<Placement> pri, X, Xe;
  for (int i = 0; i < n_priority; ++i) {
    if (priority[i].service < 0 || priority[i].service >= n_services || priority[i].server < 0 || priority[i].server > N)
      return EPARA_E_INVALID;
    pri.push_back(std::make_pair(priority[i].service, priority[i].server));
  }
  for (int l = 0; l < n_services; ++l)
    for (int n = 0; n < N; ++n) X.push_back(std::make_pair(l, n));
  for (int l = 0; l < n_services; ++l) Xe.push_back(std::make_pair(l, N));
  const std::vector<Placement> th1 = spf(phi, feas, pri, std::vector<Placement>(), false, true);    // S1: priority list
  const std::vector<Placement> th2 = spf(phi, feas, X, th1, true, false);                          // S2: real servers
  const std::vector<Placement> th3 = spf(phi, feas, Xe, th2, true, false);                         // S3: hypothetical server
  *n_out = (int)th3.size();
  if ((int)th3.size() > out_cap) return EPARA_E_RESOURCE;
  for (size_t i = 0; i < th3.size(); ++i) { out[i].service = th3[i].first; out[i].server = th3[i].second; }
  return EPARA_OK;
}

}  // extern "C"
