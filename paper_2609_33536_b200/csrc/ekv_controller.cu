// Host-side pressure-aware fidelity controller (Algorithm 1 of the paper, Sec. 3.3; state table and
// hooks of App. B.1; commit rules of App. B.2). Pure host code: it decides, the kernels in
// ekv_transition.cu move the bytes.
#include "../../include/ekv_controller.h"

#include <algorithm>
#include <map>
#include <vector>

namespace {

enum PairMode { kTarget = 0, kBase = 1, kDemoting = 2, kPromoting = 3 };

struct Pair {
    int mode = kTarget;
    int slot = -1;            // residual slot while BASE / in flight
    int new_block = -1;       // block reserved for member 1 while promoting
};

struct Request {
    int n_tokens = 0;
    int64_t last_use = 0;
    std::vector<int> blocks;  // logical -> physical; both entries of a BASE pair hold the kept block
    std::vector<Pair> pairs;  // one per two logical blocks (the last may be a lone block)
};

struct Item { int req, pair; };

} // namespace

struct ekv_ctrl {
    ekv_ctrl_config cfg{};
    std::map<int, Request> reqs;
    std::vector<int> free_blocks;     // kept sorted descending: pop_back gives the lowest id
    std::vector<int> free_slots;
    std::vector<Item> demoting, promoting;
    int64_t step = 0;
    int64_t reserve_step = -1;   // step whose reserve update (R_t) has been applied
    int reserve = 0, shortage = 0, surplus = 0, pending_surplus = 0, budget = 0, base_pairs = 0;

    int blocks_for(int n_tokens) const { return (n_tokens + cfg.page_size - 1) / cfg.page_size; }
    int take_block() { int b = free_blocks.back(); free_blocks.pop_back(); return b; }
    void give_block(int b)
    {
        free_blocks.insert(std::upper_bound(free_blocks.begin(), free_blocks.end(), b, std::greater<int>()), b);
    }
    // a pair may be demoted when both members are completely filled and it is neither a sink nor a recent pair
    bool protected_pair(const Request &r, int p) const
    {
        const int full_pairs = r.n_tokens / (2 * cfg.page_size);
        if (p >= full_pairs) return true;
        const int n_pairs = (int)r.pairs.size();
        return p < cfg.sink_pairs || p >= n_pairs - cfg.recent_pairs;
    }
};

extern "C" ekv_ctrl *ekv_ctrl_create(const ekv_ctrl_config *cfg)
{
    if (!cfg || cfg->num_blocks <= 0 || cfg->page_size <= 0 || cfg->min_demote_pairs < 0 || cfg->reserve_decay < 0 ||
        cfg->sink_pairs < 0 || cfg->recent_pairs < 0 || cfg->resid_slots < 0)
        return nullptr;
    ekv_ctrl *c = new ekv_ctrl();
    c->cfg = *cfg;
    for (int b = cfg->num_blocks - 1; b >= 0; --b) c->free_blocks.push_back(b);
    for (int s = cfg->resid_slots - 1; s >= 0; --s) c->free_slots.push_back(s);
    return c;
}

extern "C" void ekv_ctrl_destroy(ekv_ctrl *c) { delete c; }

static int grow(ekv_ctrl *c, Request &r, int new_n_tokens)
{
    if (new_n_tokens < r.n_tokens) return EKV_CTRL_ERR_ARG;
    const int need = c->blocks_for(new_n_tokens) - (int)r.blocks.size();
    if (need > (int)c->free_blocks.size()) return EKV_CTRL_ERR_NO_BLOCKS;
    for (int i = 0; i < need; ++i) r.blocks.push_back(c->take_block());
    r.pairs.resize((r.blocks.size() + 1) / 2);
    r.n_tokens = new_n_tokens;
    return EKV_CTRL_OK;
}

extern "C" int ekv_ctrl_add_request(ekv_ctrl *c, int32_t req, int32_t n_tokens)
{
    if (!c || n_tokens < 0 || c->reqs.count(req)) return EKV_CTRL_ERR_ARG;
    Request r;
    r.last_use = c->step;
    const int rc = grow(c, r, n_tokens);
    if (rc) { for (int b : r.blocks) c->give_block(b); return rc; }
    c->reqs[req] = r;
    return EKV_CTRL_OK;
}

extern "C" int ekv_ctrl_grow_request(ekv_ctrl *c, int32_t req, int32_t new_n_tokens)
{
    if (!c) return EKV_CTRL_ERR_ARG;
    auto it = c->reqs.find(req);
    if (it == c->reqs.end()) return EKV_CTRL_ERR_ARG;
    return grow(c, it->second, new_n_tokens);
}

extern "C" int ekv_ctrl_remove_request(ekv_ctrl *c, int32_t req)
{
    if (!c) return EKV_CTRL_ERR_ARG;
    auto it = c->reqs.find(req);
    if (it == c->reqs.end()) return EKV_CTRL_ERR_ARG;
    Request &r = it->second;
    for (const Pair &p : r.pairs)
        if (p.mode == kDemoting || p.mode == kPromoting) return EKV_CTRL_ERR_STATE;   // a transition is in flight
    for (size_t p = 0; p < r.pairs.size(); ++p) {
        if (r.pairs[p].mode == kBase) {
            c->give_block(r.blocks[2 * p]);                      // one physical block holds the pair
            c->free_slots.push_back(r.pairs[p].slot);
            --c->base_pairs;
        } else {
            c->give_block(r.blocks[2 * p]);
            if (2 * p + 1 < r.blocks.size()) c->give_block(r.blocks[2 * p + 1]);
        }
    }
    c->reqs.erase(it);
    return EKV_CTRL_OK;
}

extern "C" int ekv_ctrl_touch(ekv_ctrl *c, int32_t req)
{
    if (!c) return EKV_CTRL_ERR_ARG;
    auto it = c->reqs.find(req);
    if (it == c->reqs.end()) return EKV_CTRL_ERR_ARG;
    it->second.last_use = c->step;
    return EKV_CTRL_OK;
}

extern "C" int32_t ekv_ctrl_demand_for(const ekv_ctrl *c, int32_t req, int32_t new_n_tokens)
{
    if (!c) return EKV_CTRL_ERR_ARG;
    auto it = c->reqs.find(req);
    const int have = it == c->reqs.end() ? 0 : (int)it->second.blocks.size();
    return std::max(0, c->blocks_for(new_n_tokens) - have);
}

// R_t = max(0, R_{t-1} - lambda) + E_t, applied exactly once per step: by the step's promotion plan,
// or, when a step has none, when the next step begins.
static void advance_reserve(ekv_ctrl *c)
{
    if (c->reserve_step == c->step) return;
    c->reserve = std::max(0, c->reserve - c->cfg.reserve_decay) + c->pending_surplus;
    c->pending_surplus = 0;
    c->reserve_step = c->step;
}

extern "C" int ekv_ctrl_plan_demotion(ekv_ctrl *c, int32_t demand, int32_t *pair_req, int32_t *pair_idx,
                                      int32_t *resid_slot, int32_t cap, int32_t *n_out)
{
    if (!c || !n_out || demand < 0) return EKV_CTRL_ERR_ARG;
    if (!c->demoting.empty()) return EKV_CTRL_ERR_STATE;
    advance_reserve(c);             // a step that ended without a promotion plan still ages the reserve once
    ++c->step;
    *n_out = 0;
    const int free_now = (int)c->free_blocks.size();
    c->shortage = std::max(0, demand - free_now);                       // Delta_t
    if (c->shortage == 0) return EKV_CTRL_OK;
    // eligible TARGET pairs, least recently used request first, oldest pair first
    struct Cand { int64_t use; int req, pair; };
    std::vector<Cand> cand;
    for (auto &kv : c->reqs) {
        const Request &r = kv.second;
        for (int p = 0; p < (int)r.pairs.size(); ++p)
            if (r.pairs[p].mode == kTarget && !c->protected_pair(r, p)) cand.push_back({r.last_use, kv.first, p});
    }
    std::sort(cand.begin(), cand.end(), [](const Cand &a, const Cand &b) {
        if (a.use != b.use) return a.use < b.use;
        if (a.req != b.req) return a.req < b.req;
        return a.pair < b.pair;
    });
    int eligible = std::min((int)cand.size(), (int)c->free_slots.size());      // a pair needs recoverable backing
    const int n_d = std::min(eligible, std::max(c->shortage, c->cfg.min_demote_pairs));
    if (n_d > cap || (n_d > 0 && (!pair_req || !pair_idx || !resid_slot))) return EKV_CTRL_ERR_CAPACITY;
    for (int i = 0; i < n_d; ++i) {
        Request &r = c->reqs[cand[i].req];
        Pair &p = r.pairs[cand[i].pair];
        p.mode = kDemoting;
        p.slot = c->free_slots.back(); c->free_slots.pop_back();
        pair_req[i] = cand[i].req; pair_idx[i] = cand[i].pair; resid_slot[i] = p.slot;
        c->demoting.push_back({cand[i].req, cand[i].pair});
    }
    *n_out = n_d;
    c->pending_surplus = std::max(0, n_d - c->shortage);                 // E_t, recorded at commit
    return EKV_CTRL_OK;
}

extern "C" int ekv_ctrl_commit_demotion(ekv_ctrl *c, int32_t n, const int32_t *freed_blocks)
{
    if (!c || n != (int)c->demoting.size() || (n > 0 && !freed_blocks)) return c ? EKV_CTRL_ERR_STATE : EKV_CTRL_ERR_ARG;
    for (int i = 0; i < n; ++i) {
        Request &r = c->reqs[c->demoting[i].req];
        const int p = c->demoting[i].pair;
        if (r.blocks[2 * p + 1] != freed_blocks[i]) return EKV_CTRL_ERR_STATE;   // the GPU released another block
    }
    for (int i = 0; i < n; ++i) {
        Request &r = c->reqs[c->demoting[i].req];
        const int p = c->demoting[i].pair;
        c->give_block(r.blocks[2 * p + 1]);
        r.blocks[2 * p + 1] = r.blocks[2 * p];
        r.pairs[p].mode = kBase;
        ++c->base_pairs;
    }
    c->demoting.clear();
    c->surplus = c->pending_surplus;
    return EKV_CTRL_OK;
}

extern "C" int ekv_ctrl_plan_promotion(ekv_ctrl *c, int32_t transfer_slack, int32_t *pair_req, int32_t *pair_idx,
                                       int32_t *new_blocks, int32_t *resid_slot, int32_t cap, int32_t *n_out)
{
    if (!c || !n_out || transfer_slack < 0) return EKV_CTRL_ERR_ARG;
    if (!c->demoting.empty()) return EKV_CTRL_ERR_STATE;               // demotion of this step not committed yet
    *n_out = 0;
    // R_t = max(0, R_{t-1} - lambda) + E_t ;  P_t = max(0, F_post - R_t)
    advance_reserve(c);
    c->budget = std::max(0, (int)c->free_blocks.size() - c->reserve);
    int n_p = std::min(c->budget, transfer_slack);
    if (n_p == 0) return EKV_CTRL_OK;
    struct Cand { int64_t use; int req, pair; };
    std::vector<Cand> cand;
    for (auto &kv : c->reqs)
        for (int p = 0; p < (int)kv.second.pairs.size(); ++p)
            if (kv.second.pairs[p].mode == kBase) cand.push_back({kv.second.last_use, kv.first, p});
    std::sort(cand.begin(), cand.end(), [](const Cand &a, const Cand &b) {
        if (a.use != b.use) return a.use > b.use;                       // most recently used first
        if (a.req != b.req) return a.req < b.req;
        return a.pair < b.pair;
    });
    n_p = std::min(n_p, (int)cand.size());
    if (n_p > cap || (n_p > 0 && (!pair_req || !pair_idx || !new_blocks || !resid_slot))) return EKV_CTRL_ERR_CAPACITY;
    for (int i = 0; i < n_p; ++i) {
        Pair &p = c->reqs[cand[i].req].pairs[cand[i].pair];
        p.mode = kPromoting;
        p.new_block = c->take_block();                                  // reserved before the transfer starts
        pair_req[i] = cand[i].req; pair_idx[i] = cand[i].pair; new_blocks[i] = p.new_block; resid_slot[i] = p.slot;
        c->promoting.push_back({cand[i].req, cand[i].pair});
    }
    *n_out = n_p;
    return EKV_CTRL_OK;
}

extern "C" int ekv_ctrl_commit_promotion(ekv_ctrl *c, int32_t n)
{
    if (!c || n < 0 || n > (int)c->promoting.size()) return c ? EKV_CTRL_ERR_STATE : EKV_CTRL_ERR_ARG;
    for (int i = 0; i < n; ++i) {
        Request &r = c->reqs[c->promoting[i].req];
        Pair &p = r.pairs[c->promoting[i].pair];
        r.blocks[2 * c->promoting[i].pair + 1] = p.new_block;           // mapping published only now
        c->free_slots.push_back(p.slot);
        p = Pair();
        --c->base_pairs;
    }
    c->promoting.erase(c->promoting.begin(), c->promoting.begin() + n);
    return EKV_CTRL_OK;
}

extern "C" int32_t ekv_ctrl_free_blocks(const ekv_ctrl *c) { return c ? (int32_t)c->free_blocks.size() : EKV_CTRL_ERR_ARG; }
extern "C" int32_t ekv_ctrl_reserve(const ekv_ctrl *c) { return c ? c->reserve : EKV_CTRL_ERR_ARG; }
extern "C" int32_t ekv_ctrl_last_shortage(const ekv_ctrl *c) { return c ? c->shortage : EKV_CTRL_ERR_ARG; }
extern "C" int32_t ekv_ctrl_last_surplus(const ekv_ctrl *c) { return c ? c->surplus : EKV_CTRL_ERR_ARG; }
extern "C" int32_t ekv_ctrl_last_budget(const ekv_ctrl *c) { return c ? c->budget : EKV_CTRL_ERR_ARG; }
extern "C" int32_t ekv_ctrl_base_pairs(const ekv_ctrl *c) { return c ? c->base_pairs : EKV_CTRL_ERR_ARG; }

extern "C" int32_t ekv_ctrl_request_blocks(const ekv_ctrl *c, int32_t req)
{
    if (!c) return EKV_CTRL_ERR_ARG;
    auto it = c->reqs.find(req);
    return it == c->reqs.end() ? EKV_CTRL_ERR_ARG : (int32_t)it->second.blocks.size();
}

extern "C" int ekv_ctrl_block_table(const ekv_ctrl *c, int32_t req, int32_t *out, int32_t cap)
{
    if (!c || !out) return EKV_CTRL_ERR_ARG;
    auto it = c->reqs.find(req);
    if (it == c->reqs.end()) return EKV_CTRL_ERR_ARG;
    const std::vector<int> &b = it->second.blocks;
    if ((int)b.size() > cap) return EKV_CTRL_ERR_CAPACITY;
    std::copy(b.begin(), b.end(), out);
    return (int)b.size();
}

extern "C" int ekv_ctrl_pair_mode(const ekv_ctrl *c, int32_t req, int32_t pair)
{
    if (!c) return EKV_CTRL_ERR_ARG;
    auto it = c->reqs.find(req);
    if (it == c->reqs.end() || pair < 0 || pair >= (int)it->second.pairs.size()) return EKV_CTRL_ERR_ARG;
    return it->second.pairs[pair].mode;
}
