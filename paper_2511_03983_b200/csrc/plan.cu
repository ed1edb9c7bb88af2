// twist_plan_create / destroy / stats and twist_workspace_bytes: the plan object of the C ABI.
#include "plan.cuh"

#include <new>

namespace twist {

namespace {
thread_local twist_plan* t_active = nullptr;
constexpr size_t kMaxCachedMaps = 8192;      // beyond this the cache is emptied (a training loop uses a few dozen)
}  // namespace

twist_plan* active_plan() { return t_active; }

PlanScope::PlanScope(twist_plan* plan) : prev(t_active) { t_active = plan; }
PlanScope::~PlanScope() { t_active = prev; }

bool plan_lookup(const MapKey& key, CUtensorMap* map) {
  twist_plan* p = t_active;
  if (!p) return false;
  std::lock_guard<std::mutex> lock(p->mu);
  auto it = p->maps.find(key);
  if (it == p->maps.end()) {
    ++p->misses;
    return false;
  }
  ++p->hits;
  *map = it->second;
  return true;
}

void plan_store(const MapKey& key, const CUtensorMap& map) {
  twist_plan* p = t_active;
  if (!p) return;
  std::lock_guard<std::mutex> lock(p->mu);
  if (p->maps.size() >= kMaxCachedMaps) p->maps.clear();
  p->maps.emplace(key, map);
}

}  // namespace twist

extern "C" int32_t twist_plan_create(const twist_config* cfg, twist_plan** out) {
  if (!cfg || !out) return TWIST_ERR_NULL;
  *out = nullptr;
  if (cfg->struct_size != sizeof(twist_config)) return TWIST_ERR_SHAPE;
  if (cfg->n_layers <= 0 || cfg->d_model <= 0 || cfg->d_ff <= 0 || cfg->n_subnets <= 0 || cfg->tokens <= 0 ||
      cfg->ffn_block <= 0 || cfg->d_ff % cfg->ffn_block != 0 || cfg->n_heads < 0)
    return TWIST_ERR_SHAPE;
  if (cfg->n_subnets > TWIST_MAX_SUBNETS) return TWIST_ERR_UNSUPPORTED;
  if (cfg->ffn_kind < TWIST_FFN_RELU || cfg->ffn_kind > TWIST_FFN_SWIGLU) return TWIST_ERR_SHAPE;
  if (cfg->dtype != TWIST_FP32 && cfg->dtype != TWIST_BF16) return TWIST_ERR_SHAPE;
  const int nb = cfg->d_ff / cfg->ffn_block;
  if (cfg->ffn_keep <= 0 || cfg->ffn_keep > nb) return TWIST_ERR_INFEASIBLE;
  if (cfg->n_heads > 0) {
    if (cfg->n_kv_heads <= 0 || cfg->n_heads % cfg->n_kv_heads != 0 || cfg->d_head <= 0) return TWIST_ERR_SHAPE;
    if (cfg->head_keep <= 0 || cfg->head_keep > cfg->n_heads) return TWIST_ERR_INFEASIBLE;
  }
  twist_plan* p = new (std::nothrow) twist_plan();      // host memory only
  if (!p) return TWIST_ERR_WORKSPACE;
  p->cfg = *cfg;
  *out = p;
  return TWIST_OK;
}

extern "C" int32_t twist_plan_destroy(twist_plan* plan) {
  if (!plan) return TWIST_ERR_NULL;
  delete plan;
  return TWIST_OK;
}

extern "C" int32_t twist_plan_stats(twist_plan* plan, uint64_t* cached, uint64_t* hits, uint64_t* misses) {
  if (!plan) return TWIST_ERR_NULL;
  std::lock_guard<std::mutex> lock(plan->mu);
  if (cached) *cached = plan->maps.size();
  if (hits) *hits = plan->hits;
  if (misses) *misses = plan->misses;
  return TWIST_OK;
}

extern "C" int32_t twist_workspace_bytes(const twist_plan* plan, size_t* bytes) {
  if (!plan || !bytes) return TWIST_ERR_NULL;
  const twist_config& c = plan->cfg;
  const int S = c.n_subnets, T = c.tokens, d = c.d_model;
  int widest = d;                                        // output widths of the blocks a loss can sit on
  if (c.n_heads > 0) {
    const int kv_max = c.n_kv_heads < c.head_keep ? c.n_kv_heads : c.head_keep;
    const int nq = (c.head_keep + 2 * kv_max) * c.d_head;
    const int nq_full = (c.n_heads + 2 * c.n_kv_heads) * c.d_head;      // shared layers, masked workers
    widest = widest > nq ? widest : nq;
    widest = widest > nq_full ? widest : nq_full;
  }
  size_t need = twist_mse_workspace_bytes(S);
  const size_t fused = twist_fused_loss_workspace_bytes(S, T, widest);
  const size_t ln = twist_layernorm_workspace_bytes(S, T, d);
  need = need > fused ? need : fused;
  need = need > ln ? need : ln;
  *bytes = need;
  return TWIST_OK;
}
