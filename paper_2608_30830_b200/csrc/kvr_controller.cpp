// Live retention controller: the paper's two-stage policy driven by a clock, on top of the pool's C ABI.
// Host code only; every byte it causes to move goes through kvr_suspend_to_host / kvr_resume_from_host.
#include <cmath>
#include <cstdint>
#include <limits>
#include <map>
#include <set>
#include <unordered_map>
#include <utility>

#include "../../include/kvr.h"

namespace {
constexpr double kInf = std::numeric_limits<double>::infinity();
enum Where { IN_HBM = 1, ON_HOST = 2, GONE = 3 };
struct Ctx {
  int where = 0;
  double suspended_at = 0;   // also the recency key: the longest-suspended context is evicted first
  double deadline = kInf;    // offload deadline while IN_HBM, expiry deadline while ON_HOST
};
}  // namespace

struct kvr_controller {
  kvr_pool *pool = nullptr;
  kvr_controller_config cfg{};
  double c2 = 0, t2 = kInf, now = -kInf;
  std::unordered_map<uint64_t, Ctx> ctx;
  std::set<std::pair<double, uint64_t>> timers;   // (deadline, request): offload or expiry, by Ctx::where
  std::set<std::pair<double, uint64_t>> lru;      // (suspended_at, request) of contexts on the host
  kvr_controller_stats st{};

  void arm(uint64_t id, Ctx &c, double deadline) {
    c.deadline = deadline;
    if (deadline < kInf) timers.insert({deadline, id});
  }
  void disarm(uint64_t id, Ctx &c) {
    if (c.deadline < kInf) timers.erase({c.deadline, id});
    c.deadline = kInf;
  }
  void to_gone(uint64_t id, Ctx &c) {
    disarm(id, c);
    if (c.where == ON_HOST) lru.erase({c.suspended_at, id});
    c.where = GONE;
  }
  // state 1 -> 2; on a full tier apply the admission rule.  Returns KVR_OK or KVR_HOST_FULL (context discarded).
  kvr_status offload(uint64_t id, Ctx &c) {
    disarm(id, c);
    for (;;) {
      kvr_status s = kvr_suspend_to_host(pool, &id, 1, 0, nullptr);
      if (s == KVR_OK) break;
      if (s != KVR_HOST_FULL) return s;
      // live rule, first class (Appendix D: "blocks whose timer has expired" go first): a host copy whose one-shot
      // timer has run out by this instant but has not been fired yet (it is due at the very same time as this
      // offload) is discarded before any copy that is still within its timer
      if (cfg.admission == KVR_ADMIT_LIVE) {
        uint64_t due = 0;
        bool found = false;
        for (auto it = timers.begin(); it != timers.end() && it->first <= now; ++it)
          if (ctx[it->second].where == ON_HOST) { due = it->second; found = true; break; }
        if (found) {
          Ctx &v = ctx[due];
          kvr_status e = kvr_expire(pool, &due, 1, nullptr);
          if (e != KVR_OK) return e;
          to_gone(due, v);
          st.ttl_expired++;
          continue;
        }
      }
      // the paper's second class, transient blocks of active requests, has no counterpart here: the host tier holds
      // images of suspended contexts only.  Third class: the least recently suspended host copy.
      // Replay rule: never displace.
      if (cfg.admission == KVR_ADMIT_LIVE && !lru.empty()) {
        const uint64_t victim = lru.begin()->second;
        Ctx &v = ctx[victim];
        kvr_status e = kvr_expire(pool, &victim, 1, nullptr);
        if (e != KVR_OK) return e;
        to_gone(victim, v);
        st.evicted_lru++;
        continue;
      }
      kvr_status e = kvr_expire(pool, &id, 1, nullptr);        // not admitted: recompute at resume
      if (e != KVR_OK) return e;
      st.gpu_cost += cfg.prices.alpha1 * (now - c.suspended_at);   // HBM time it did use
      c.where = GONE;
      st.not_admitted++;
      return KVR_HOST_FULL;
    }
    st.gpu_cost += cfg.prices.alpha1 * (now - c.suspended_at);
    c.where = ON_HOST;
    lru.insert({c.suspended_at, id});
    st.offloaded++;
    if (cfg.branch == KVR_BRANCH_TTL) arm(id, c, now + t2);        // one-shot timer, counted from the offload
    return KVR_OK;
  }
  kvr_status advance(double t, int32_t *n_off, int32_t *n_exp) {
    if (!(t >= now)) return KVR_ERR_INVALID_ARG;
    while (!timers.empty() && timers.begin()->first <= t) {
      const auto [deadline, id] = *timers.begin();
      now = deadline > now ? deadline : now;
      Ctx &c = ctx[id];
      if (c.where == IN_HBM) {
        kvr_status s = offload(id, c);
        if (s < 0) return s;
        if (s == KVR_OK && n_off) ++*n_off;
      } else {                                                     // ON_HOST: the timer fires, the copy is discarded
        kvr_status e = kvr_expire(pool, &id, 1, nullptr);
        if (e != KVR_OK) return e;
        to_gone(id, c);
        st.ttl_expired++;
        if (n_exp) ++*n_exp;
      }
    }
    now = t;
    return KVR_OK;
  }
};

extern "C" {

kvr_status kvr_controller_create(kvr_pool *pool, const kvr_controller_config *cfg, kvr_controller **out) {
  if (!pool || !cfg || !out) return KVR_ERR_INVALID_ARG;
  double t1, ts;
  if (kvr_policy_break_evens(&cfg->prices, &t1, &ts) != KVR_OK) return KVR_ERR_INVALID_ARG;
  if (cfg->branch != KVR_BRANCH_RETAIN && cfg->branch != KVR_BRANCH_TTL) return KVR_ERR_INVALID_ARG;
  if (cfg->admission != KVR_ADMIT_REPLAY && cfg->admission != KVR_ADMIT_LIVE) return KVR_ERR_INVALID_ARG;
  if (!(cfg->hbm_grace_s >= 0) || !(cfg->w_ref > 0) || !(cfg->lambda >= 0)) return KVR_ERR_INVALID_ARG;
  double c2 = cfg->c2;
  if (!(c2 > 0)) {
    if (!(cfg->mean_image_bytes > 0)) return KVR_ERR_INVALID_ARG;
    kvr_stats s;
    if (kvr_status e = kvr_pool_stats(pool, &s)) return e;
    c2 = (double)s.host_capacity / cfg->mean_image_bytes;
    if (!(c2 > 0)) return KVR_ERR_INVALID_ARG;
  }
  kvr_controller *c = new (std::nothrow) kvr_controller();
  if (!c) return KVR_ERR_NOMEM;
  c->pool = pool; c->cfg = *cfg; c->c2 = c2;
  if (kvr_status e = kvr_policy_host_ttl(&cfg->prices, cfg->lambda, c2, cfg->w_ref, nullptr, &c->t2)) { delete c; return e; }
  c->st.t2 = c->t2; c->st.branch = cfg->branch;
  *out = c;
  return KVR_OK;
}

kvr_status kvr_controller_destroy(kvr_controller *c) { delete c; return KVR_OK; }

kvr_status kvr_controller_calibrate(kvr_controller *c, const double *arrive, const double *wait, int64_t n, int32_t *branch) {
  if (!c) return KVR_ERR_INVALID_ARG;
  int32_t use_ttl = 0;
  const int64_t slots = (int64_t)std::floor(c->c2);
  if (kvr_status e = kvr_policy_select(&c->cfg.prices, arrive, wait, n, c->cfg.lambda, slots > 0 ? slots : 1, c->cfg.w_ref,
                                       &use_ttl, nullptr, nullptr, nullptr)) return e;
  c->cfg.branch = use_ttl ? KVR_BRANCH_TTL : KVR_BRANCH_RETAIN;   // frozen for the run that follows
  c->st.branch = c->cfg.branch;
  if (branch) *branch = c->cfg.branch;
  return KVR_OK;
}

kvr_status kvr_controller_advance(kvr_controller *c, double now, int32_t *n_offloaded, int32_t *n_expired) {
  if (!c) return KVR_ERR_INVALID_ARG;
  if (n_offloaded) *n_offloaded = 0;
  if (n_expired) *n_expired = 0;
  return c->advance(now, n_offloaded, n_expired);
}

kvr_status kvr_controller_suspend(kvr_controller *c, uint64_t req, double now) {
  if (!c) return KVR_ERR_INVALID_ARG;
  if (kvr_status e = c->advance(now, nullptr, nullptr)) return e;
  auto it = c->ctx.find(req);
  if (it != c->ctx.end() && it->second.where != GONE) return KVR_ERR_BAD_STATE;
  kvr_status s = kvr_retain_in_hbm(c->pool, &req, 1, nullptr);   // suspension: the context is pinned where it is
  if (s != KVR_OK) return s;
  Ctx &x = c->ctx[req];
  x = Ctx();
  x.where = IN_HBM; x.suspended_at = now;
  c->st.suspended++;
  if (c->cfg.hbm_grace_s > 0) { c->arm(req, x, now + c->cfg.hbm_grace_s); return KVR_RESIDENT; }
  return c->offload(req, x);
}

kvr_status kvr_controller_resume(kvr_controller *c, uint64_t req, double now) {
  if (!c) return KVR_ERR_INVALID_ARG;
  if (kvr_status e = c->advance(now, nullptr, nullptr)) return e;
  auto it = c->ctx.find(req);
  if (it == c->ctx.end()) return KVR_ERR_UNKNOWN_REQUEST;
  Ctx &x = it->second;
  kvr_status s = kvr_resume_from_host(c->pool, &req, 1, 0, nullptr);
  if (s == KVR_HBM_FULL || s < 0) return s;                      // nothing changed; the caller frees blocks and retries
  if (s == KVR_RESIDENT) { c->st.gpu_cost += c->cfg.prices.alpha1 * (now - x.suspended_at); c->st.resumed_hbm++; c->disarm(req, x); }
  else if (s == KVR_OK) { c->st.gpu_cost += c->cfg.prices.beta2; c->st.resumed_host++; c->disarm(req, x); c->lru.erase({x.suspended_at, req}); }
  else { c->st.gpu_cost += c->cfg.prices.beta3; c->st.recomputed++; }
  c->ctx.erase(it);
  return s;
}

kvr_status kvr_controller_get_stats(kvr_controller *c, kvr_controller_stats *out) {
  if (!c || !out) return KVR_ERR_INVALID_ARG;
  *out = c->st;
  out->tracked = (int64_t)c->ctx.size();
  return KVR_OK;
}

}  // extern "C"
