// kvt_oracle.cpp — plain, slow, single-threaded CPU statement of what the KV-cache hot path computes.
//
// THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT. Only the tests, the smoke check and the
// benchmark's CPU-baseline leg may load it. It shares no code with the CUDA library: its own
// hash, its own containers (std::map / std::set / std::vector), its own payload copies.
// All pointers are ordinary host memory.
//
// What each part follows:
//   - message-level primitives and their effect on per-context message states: Table 3,
//     Section 5.1 (KV scope resolution: suffix invalidation, KV-existence gating, program order)
//     and Section 5.2 (runtime transitions; remove/replace; fork; one_off);
//   - KV-level state of a shared block = highest-priority mapped message state, dead when every
//     mapped version is Discarded: Section 6.1 (KV shared between contexts);
//   - release order Expired/Temporary -> Suspended -> Active and "admit iff Delta <= 0":
//     Algorithm 1; most-recently-suspended-first inside the Suspended tier: Section 6.2; the
//     oldest-first switch is the "w/o RO" variant of Section 8.3;
//   - two tiers (HBM, host) with byte-for-byte block movement: Section 7.
// The paper does not define a block hash, a block size, tie-breaks or slot assignment; the readings
// used here (chained 64-bit hash over 16-token blocks, lowest-free-slot-first, depth-descending then
// slot-ascending ties, logical clock) are listed in the repository's design notes.
//
// What holds this file to the paper and to arithmetic, independently of the CUDA library (CPU-only tests):
// the published SplitMix64 output stream for the mixing function and the lane multipliers; the closed
// form and the affine-composition law of the chain; prefix / suffix invariants; the literal double loop
// of Section 6.1 (kvto_classify_bruteforce) and a brute-force victim sort on tiny pools; the paper's
// shared-KV example; Algorithm 1's order; LRU / reverse-LRU special cases; byte-identical round trips;
// hand-worked scenarios for the destination slots of offload / move and for the recency stamps of a
// call that ends in flight. Every function is covered by at least one of these.

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <map>
#include <set>
#include <string>
#include <thread>
#include <utility>
#include <vector>

namespace {

enum : int32_t {
  OK = 0, E_INVAL = -1, E_NOCTX = -2, E_RANGE = -3, E_STATE = -4, E_NOSPACE = -5, E_BUFSZ = -6
};
enum : uint32_t { TIER_HBM = 0, TIER_HOST = 1, TIER_REMOTE = 2, N_TIERS = 3 };
enum : uint32_t { LAYOUT_LAYER_MAJOR = 0, LAYOUT_BLOCK_MAJOR = 1 };
enum : uint32_t { ORDER_MRU = 0, ORDER_LRU = 1 };
enum : uint32_t {
  POLICY_NO_LIFECYCLE = 1,   // the "w/o LT" variant of Section 8.3
  POLICY_ORPHANS_DEAD = 4,   // a context's mappings stop counting at its first non-resident block
  POLICY_INCLUSIVE = 2       // a reloaded block keeps its host copy (Section 7: a tier may keep a copy of a page that has moved on)
};
enum : uint32_t {
  OP_SPAWN = 1, OP_FORK, OP_APPEND, OP_REPLACE, OP_REMOVE, OP_ONE_OFF, OP_PREFILL_DONE,
  OP_TERMINATE, OP_PIN, OP_UNPIN
};
// message-level states (Section 5.2)
enum : uint8_t { MS_ACTIVE = 0, MS_SUSPENDED = 1, MS_EXPIRED = 2, MS_TEMPORARY = 3, MS_PINNED = 4 };

// Priority of a message state for the block aggregate, following Algorithm 1's release order:
// Discarded (Expired, Temporary) lowest, then Suspended, then Active, then Pinned.
int msgrank(uint8_t s) {
  switch (s) {
    case MS_PINNED: return 3;
    case MS_ACTIVE: return 2;
    case MS_SUSPENDED: return 1;
    default: return 0;
  }
}

// ---- block hash -------------------------------------------------------------------------------
// mix64 is the SplitMix64 output function (a bijection on 64-bit words).
uint64_t mix64(uint64_t z) {
  z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull;
  z ^= z >> 27; z *= 0x94D049BB133111EBull;
  z ^= z >> 31;
  return z;
}
const uint64_t GOLD = 0x9E3779B97F4A7C15ull;

struct HashParams { uint64_t K[16]; uint64_t P; uint64_t H0; };

HashParams make_params(uint64_t seed) {
  HashParams p;
  for (int t = 0; t < 16; ++t) p.K[t] = mix64(GOLD * (uint64_t)(t + 1)) | 1ull;
  p.P = mix64(GOLD * 17ull) | 1ull;
  p.H0 = mix64(seed ^ (GOLD * 18ull));
  return p;
}

// key_b for every full 16-token block, by the definition: a plain loop over blocks.
void hash_blocks(const HashParams &hp, const uint32_t *tok, uint64_t T, std::vector<uint64_t> &keys) {
  uint64_t nb = T / 16;
  keys.resize(nb);
  uint64_t h = hp.H0;
  for (uint64_t b = 0; b < nb; ++b) {
    uint64_t s = 0;
    for (int t = 0; t < 16; ++t) s += ((uint64_t)tok[16 * b + t] + 1ull) * hp.K[t];
    uint64_t d = mix64(s);
    h = hp.P * h + d;
    uint64_t key = mix64(h);
    if (key < 2) key += 2;
    keys[b] = key;
  }
}

// ---- engine -------------------------------------------------------------------------------------
struct Msg { std::vector<uint32_t> tok; uint8_t state; };

struct Ctx {
  bool live = false;
  bool terminated = false;   // ended, but kept because it still has Pinned messages (Section 5.2)
  std::vector<Msg> msgs;
  bool one_off = false, in_flight = false;
  // materialised mapping: token sequence as of the last call (or inherited at fork), the bounds of
  // the leading messages whose positions in it are still valid, and its block keys.
  std::vector<uint32_t> mat_tokens;
  std::vector<std::pair<uint32_t, uint32_t>> mat_bounds;  // size = mat_msgs
  std::vector<uint64_t> mat_keys;                          // hash of mat_tokens
  uint32_t valid_blocks = 0;  // leading blocks of mat_keys this context still maps
  uint32_t held = 0;          // leading blocks locked in flight
  uint32_t hit_len = 0, n_hit_hbm = 0, n_hit_host = 0, n_hit_remote = 0, n_admissible = 0, n_pinned = 0;
};

struct Entry {
  uint64_t key = 0; uint32_t stamp = 0, depth = 0, inflight = 0; uint8_t floor = 0;
  // inclusive tiering: an HBM block and its clean host copy ("shadow") point at each other by slot
  int64_t link = -1;
  bool shadow = false;   // host slot that only holds a copy of a block whose home is in HBM
};

struct Config {
  uint32_t n_layers, n_kv_heads, head_dim, elem_bytes, pool_layout;
  uint32_t n_hbm_blocks, n_host_blocks, max_contexts, suspended_order, policy_flags;
  uint64_t hash_seed;
  uint8_t *hbm_pool; uint8_t *host_pool;  // host memory; NULL = metadata only
  uint32_t n_remote_blocks, pad;          // third tier (Section 7: remote memory), stood in for by one more buffer
  uint8_t *remote_pool;
};

struct CallInfo { uint32_t n_blocks, hit_len, n_hit_hbm, n_hit_host, n_admissible, n_admitted, n_held, n_pinned, n_hit_remote; };

struct Stats {
  uint64_t clock, n_contexts, occ_hbm, occ_host, blocks_hashed, hits_hbm, hits_host, misses,
      inserted, adopted, dropped, offloaded, reloaded, compacted, bytes_d2h, bytes_h2d, bytes_d2d,
      table_rebuilds, tombstones, kernel_launches, mover_launches, mover_ns, mover_bytes, lookup_ns,
      lookup_blocks, select_ns, select_slots, offloaded_clean, blocks_rehashed, occ_remote, hits_remote, demoted,
      promoted, classify_ns, classify_items;
};

struct Op {
  uint32_t op, ctx, parent, msg_start, msg_end, n_tokens, flags, reserved;
  const uint32_t *tokens;
};

struct Engine {
  Config cfg;
  HashParams hp;
  uint64_t chunk_bytes, n_chunks, block_bytes;
  std::vector<Ctx> ctxs;
  std::vector<Entry> ent[N_TIERS];          // per tier, indexed by slot; key == 0 means free
  std::set<uint32_t> free_slots[N_TIERS];   // lowest-numbered free slot first
  std::map<uint64_t, std::pair<uint32_t, uint32_t>> where;  // key -> (tier, slot)
  uint32_t now = 0;
  Stats st{};
};

uint32_t tier_size(const Engine &e, uint32_t t) {
  return t == TIER_HBM ? e.cfg.n_hbm_blocks : t == TIER_HOST ? e.cfg.n_host_blocks : e.cfg.n_remote_blocks;
}

uint8_t *chunk_ptr(const Engine &e, uint32_t tier, uint32_t slot, uint64_t c) {
  if (tier == TIER_HBM && e.cfg.pool_layout == LAYOUT_LAYER_MAJOR)
    return e.cfg.hbm_pool + (c * (uint64_t)e.cfg.n_hbm_blocks + slot) * e.chunk_bytes;
  uint8_t *base = tier == TIER_HBM ? e.cfg.hbm_pool : tier == TIER_HOST ? e.cfg.host_pool : e.cfg.remote_pool;
  return base + (uint64_t)slot * e.block_bytes + c * e.chunk_bytes;
}

void copy_payload(Engine &e, uint32_t st, uint32_t ss, uint32_t dt, uint32_t ds) {
  if (!e.cfg.hbm_pool) return;  // metadata-only engine
  for (uint64_t c = 0; c < e.n_chunks; ++c)
    std::memcpy(chunk_ptr(e, dt, ds, c), chunk_ptr(e, st, ss, c), e.chunk_bytes);
}

Ctx *get_ctx(Engine &e, uint32_t id, bool allow_terminated = false) {
  if (id >= e.ctxs.size() || !e.ctxs[id].live) return nullptr;
  if (e.ctxs[id].terminated && !allow_terminated) return nullptr;
  return &e.ctxs[id];
}

Entry *find_entry(Engine &e, uint64_t key) {
  auto it = e.where.find(key);
  if (it == e.where.end()) return nullptr;
  return &e.ent[it->second.first][it->second.second];
}

void free_slot(Engine &e, uint32_t tier, uint32_t slot) {
  Entry &x = e.ent[tier][slot];
  if (x.shadow) {                      // dropping a host copy: the block lives on in HBM
    e.ent[TIER_HBM][x.link].link = -1;
  } else {
    e.where.erase(x.key);
    if (x.link >= 0) {                 // dropping a block that has a host copy: the copy goes too
      e.ent[TIER_HOST][x.link] = Entry();
      e.free_slots[TIER_HOST].insert((uint32_t)x.link);
    }
  }
  x = Entry();
  e.free_slots[tier].insert(slot);
}

// Per-block rank of a context under a given message layout: max over the messages whose token span
// intersects the block (a block straddling several messages takes the highest of them).
void block_ranks(const Ctx &c, const std::vector<std::pair<uint32_t, uint32_t>> &bounds, uint32_t n_blocks,
                 std::vector<uint8_t> &out) {
  out.assign(n_blocks, 0);
  for (size_t j = 0; j < bounds.size(); ++j) {
    uint32_t s = bounds[j].first, t = bounds[j].second;
    if (t <= s) continue;  // empty message covers nothing
    int r = msgrank(c.msgs[j].state);
    for (uint32_t b = s / 16; b <= (t - 1) / 16 && b < n_blocks; ++b)
      if (r > out[b]) out[b] = (uint8_t)r;
  }
}

// KV-level state of every resident block (Section 6.1): the highest-priority state over all
// mappings (context c, block b < valid_blocks, same key); dead if nobody maps it. `floor` is the
// anonymous mapping installed by the debug loader.
void classify(Engine &e, std::vector<uint8_t> rank[N_TIERS]) {
  for (int t = 0; t < (int)N_TIERS; ++t) {
    rank[t].assign(e.ent[t].size(), 0xFF);
    for (size_t s = 0; s < e.ent[t].size(); ++s)
      if (e.ent[t][s].key) rank[t][s] = e.ent[t][s].shadow ? 0xFE : e.ent[t][s].floor;
  }
  std::vector<uint8_t> br;
  for (const Ctx &c : e.ctxs) {
    if (!c.live) continue;
    block_ranks(c, c.mat_bounds, c.valid_blocks, br);
    for (uint32_t b = 0; b < c.valid_blocks; ++b) {
      auto it = e.where.find(c.mat_keys[b]);
      if (it == e.where.end()) {
        if (e.cfg.policy_flags & POLICY_ORPHANS_DEAD) break;   // nothing behind a missing block is reachable
        continue;
      }
      uint8_t &r = rank[it->second.first][it->second.second];
      if (br[b] > r) r = br[b];
    }
  }
}

void unlock_held(Engine &e, Ctx &c, bool stamp) {
  for (uint32_t b = 0; b < c.held; ++b) {
    Entry *x = find_entry(e, c.mat_keys[b]);
    if (!x) continue;  // cannot happen: in-flight blocks are never evicted
    if (x->inflight) x->inflight -= 1;
    if (stamp) x->stamp = e.now;
  }
  c.held = 0;
}

// Edit at message s (remove / replace): the context stops mapping everything from the block that
// contains the first token of message s (Section 5.1, prefix-dependent validity).
void cut_at(Ctx &c, uint32_t s) {
  if (s < c.mat_bounds.size()) {
    uint32_t cut = c.mat_bounds[s].first / 16;
    if (cut < c.valid_blocks) c.valid_blocks = cut;
    c.mat_bounds.resize(s);
  }
}

}  // namespace

extern "C" {

int32_t kvto_create(const Config *cfg, Engine **out) {
  if (!cfg || !out) return E_INVAL;
  if (!cfg->n_layers || !cfg->n_kv_heads || !cfg->head_dim || !cfg->elem_bytes || !cfg->n_hbm_blocks ||
      !cfg->max_contexts || cfg->pool_layout > 1 || cfg->suspended_order > 1 || cfg->policy_flags > 7)
    return E_INVAL;
  Engine *e = new Engine();
  e->cfg = *cfg;
  e->hp = make_params(cfg->hash_seed);
  e->chunk_bytes = 16ull * cfg->n_kv_heads * cfg->head_dim * cfg->elem_bytes;
  e->n_chunks = 2ull * cfg->n_layers;
  e->block_bytes = e->chunk_bytes * e->n_chunks;
  e->ctxs.resize(cfg->max_contexts);
  e->ent[0].resize(cfg->n_hbm_blocks);
  e->ent[1].resize(cfg->n_host_blocks);
  e->ent[2].resize(cfg->n_remote_blocks);
  for (uint32_t s = 0; s < cfg->n_hbm_blocks; ++s) e->free_slots[0].insert(s);
  for (uint32_t s = 0; s < cfg->n_host_blocks; ++s) e->free_slots[1].insert(s);
  for (uint32_t s = 0; s < cfg->n_remote_blocks; ++s) e->free_slots[2].insert(s);
  *out = e;
  return OK;
}

int32_t kvto_destroy(Engine *e) { delete e; return OK; }

// Block keys of one token sequence, without an engine.
int32_t kvto_hash_tokens(const uint32_t *tokens, uint64_t n_tokens, uint64_t seed, uint64_t *keys) {
  if ((!tokens && n_tokens) || (!keys && n_tokens >= 16)) return E_INVAL;
  HashParams hp = make_params(seed);
  std::vector<uint64_t> k;
  hash_blocks(hp, tokens, n_tokens, k);
  if (!k.empty()) std::memcpy(keys, k.data(), k.size() * 8);
  return OK;
}

// The hash constants, for the pins: out[0..15] = K, out[16] = P, out[17] = H0, out[18] = mix64(x).
int32_t kvto_hash_constants(uint64_t seed, uint64_t x, uint64_t *out) {
  HashParams hp = make_params(seed);
  for (int t = 0; t < 16; ++t) out[t] = hp.K[t];
  out[16] = hp.P; out[17] = hp.H0; out[18] = mix64(x);
  return OK;
}

int32_t kvto_apply_op(Engine *e, const Op *op) {
  if (!e || !op) return E_INVAL;
  const uint32_t id = op->ctx;
  switch (op->op) {
    case OP_SPAWN: {
      if (id >= e->ctxs.size() || e->ctxs[id].live) return E_INVAL;
      e->ctxs[id] = Ctx();
      e->ctxs[id].live = true;
      return OK;
    }
    case OP_FORK: {
      if (id >= e->ctxs.size() || e->ctxs[id].live) return E_INVAL;
      Ctx *p = get_ctx(*e, op->parent);
      if (!p) return E_NOCTX;
      if (p->in_flight) return E_STATE;
      if (op->msg_end > p->msgs.size()) return E_RANGE;
      Ctx k;
      k.live = true;
      // inherited messages are newly appended to the child: Active (Section 5.2)
      for (uint32_t j = 0; j < op->msg_end; ++j) k.msgs.push_back(Msg{p->msgs[j].tok, MS_ACTIVE});
      uint32_t m = std::min<uint32_t>(op->msg_end, (uint32_t)p->mat_bounds.size());
      uint32_t T = m ? p->mat_bounds[m - 1].second : 0;
      k.mat_tokens.assign(p->mat_tokens.begin(), p->mat_tokens.begin() + T);
      k.mat_bounds.assign(p->mat_bounds.begin(), p->mat_bounds.begin() + m);
      hash_blocks(e->hp, k.mat_tokens.data(), k.mat_tokens.size(), k.mat_keys);
      k.valid_blocks = std::min<uint32_t>(T / 16, p->valid_blocks);
      e->ctxs[id] = std::move(k);
      return OK;
    }
    default: break;
  }
  if (op->op == 0 || op->op > OP_UNPIN) return E_INVAL;
  Ctx *c = get_ctx(*e, id, op->op == OP_UNPIN);   // a terminated context with Pinned messages only accepts unpin
  if (!c) return E_NOCTX;
  switch (op->op) {
    case OP_APPEND: {
      if (c->in_flight) return E_STATE;
      if (op->n_tokens && !op->tokens) return E_INVAL;
      Msg m;
      m.tok.assign(op->tokens, op->tokens + op->n_tokens);
      m.state = c->one_off ? MS_TEMPORARY : MS_ACTIVE;
      c->msgs.push_back(std::move(m));
      return OK;
    }
    case OP_REPLACE:
    case OP_REMOVE: {
      if (c->in_flight) return E_STATE;
      if (!(op->msg_start < op->msg_end && op->msg_end <= c->msgs.size())) return E_RANGE;
      if (op->op == OP_REPLACE && op->n_tokens && !op->tokens) return E_INVAL;
      cut_at(*c, op->msg_start);
      c->msgs.erase(c->msgs.begin() + op->msg_start, c->msgs.begin() + op->msg_end);
      if (op->op == OP_REPLACE) {
        Msg m;
        m.tok.assign(op->tokens, op->tokens + op->n_tokens);
        m.state = c->one_off ? MS_TEMPORARY : MS_ACTIVE;
        c->msgs.insert(c->msgs.begin() + op->msg_start, std::move(m));
      }
      return OK;
    }
    case OP_ONE_OFF: {
      if (c->in_flight) return E_STATE;
      if (op->msg_start == 0 && op->msg_end == 0xFFFFFFFFu) {
        c->one_off = true;
        for (Msg &m : c->msgs)
          if (m.state != MS_PINNED) m.state = MS_TEMPORARY;   // explicit protection stays
        return OK;
      }
      if (!(op->msg_start < op->msg_end && op->msg_end <= c->msgs.size())) return E_RANGE;
      for (uint32_t j = op->msg_start; j < op->msg_end; ++j) c->msgs[j].state = MS_TEMPORARY;
      return OK;
    }
    case OP_PREFILL_DONE: {
      if (!c->in_flight) return E_STATE;
      e->now += 1;
      unlock_held(*e, *c, true);
      for (Msg &m : c->msgs)
        if (m.state == MS_ACTIVE) m.state = MS_SUSPENDED;
      c->in_flight = false;
      return OK;
    }
    case OP_TERMINATE: {
      if (c->in_flight) unlock_held(*e, *c, false);
      bool pinned = false;
      for (Msg &m : c->msgs) {
        if (m.state == MS_PINNED) pinned = true;
        else m.state = MS_EXPIRED;   // ordinary messages expire
      }
      if (pinned) {                  // Pinned messages retain their declared protection
        c->terminated = true;
        c->in_flight = false;
      } else {
        *c = Ctx();                  // the context maps nothing any more
      }
      return OK;
    }
    case OP_PIN: {
      if (c->in_flight) return E_STATE;
      if (!(op->msg_start < op->msg_end && op->msg_end <= c->msgs.size())) return E_RANGE;
      for (uint32_t j = op->msg_start; j < op->msg_end; ++j) c->msgs[j].state = MS_PINNED;
      return OK;
    }
    case OP_UNPIN: {
      if (c->in_flight) return E_STATE;
      if (!(op->msg_start < op->msg_end && op->msg_end <= c->msgs.size())) return E_RANGE;
      // back to Suspended between calls, or to Expired if the context has terminated
      for (uint32_t j = op->msg_start; j < op->msg_end; ++j)
        if (c->msgs[j].state == MS_PINNED)
          c->msgs[j].state = c->terminated ? MS_EXPIRED : (c->one_off ? MS_TEMPORARY : MS_SUSPENDED);
      if (c->terminated) {
        bool pinned = false;
        for (const Msg &m : c->msgs) pinned = pinned || m.state == MS_PINNED;
        if (!pinned) *c = Ctx();
      }
      return OK;
    }
  }
  return E_INVAL;
}

int32_t kvto_map_blocks(Engine *e, const uint32_t *ids, uint32_t n_ctx, uint32_t phase, CallInfo *out) {
  if (!e || !ids || !out || n_ctx == 0 || phase > 1) return E_INVAL;
  for (uint32_t i = 0; i < n_ctx; ++i) {
    if (!get_ctx(*e, ids[i])) return E_NOCTX;
  }
  for (uint32_t i = 0; i < n_ctx; ++i)
    for (uint32_t j = 0; j < i; ++j)
      if (ids[i] == ids[j]) return E_INVAL;
  for (uint32_t i = 0; i < n_ctx; ++i) {
    Ctx &c = e->ctxs[ids[i]];
    if (phase == 0 && c.in_flight) return E_STATE;
    if (phase == 1 && !c.in_flight) return E_STATE;
  }
  if (phase == 0) {
    e->now += 1;
    for (uint32_t i = 0; i < n_ctx; ++i) {
      Ctx &c = e->ctxs[ids[i]];
      // the next request reactivates participating ordinary messages (Section 5.2)
      for (Msg &m : c.msgs)
        if (m.state == MS_SUSPENDED) m.state = MS_ACTIVE;
      c.in_flight = true;
      // new token layout = concatenation of the messages
      c.mat_tokens.clear();
      c.mat_bounds.clear();
      for (const Msg &m : c.msgs) {
        uint32_t s = (uint32_t)c.mat_tokens.size();
        c.mat_tokens.insert(c.mat_tokens.end(), m.tok.begin(), m.tok.end());
        c.mat_bounds.push_back({s, (uint32_t)c.mat_tokens.size()});
      }
      hash_blocks(e->hp, c.mat_tokens.data(), c.mat_tokens.size(), c.mat_keys);
      uint32_t nb = (uint32_t)c.mat_keys.size();
      c.valid_blocks = nb;
      // reusable prefix: walk the chain until the first block that is not resident
      uint32_t h = 0;
      c.n_hit_hbm = c.n_hit_host = c.n_hit_remote = 0;
      while (h < nb) {
        auto it = e->where.find(c.mat_keys[h]);
        if (it == e->where.end()) break;
        Entry &x = e->ent[it->second.first][it->second.second];
        x.stamp = e->now;
        x.inflight += 1;
        if (it->second.first == TIER_HBM) c.n_hit_hbm++;
        else if (it->second.first == TIER_HOST) c.n_hit_host++;
        else c.n_hit_remote++;
        ++h;
      }
      c.hit_len = h;
      c.held = h;
      // admissible run: up to the first block made only of Temporary tokens (Algorithm 1 bypass)
      std::vector<uint8_t> br;
      block_ranks(c, c.mat_bounds, nb, br);
      uint32_t a = h;
      c.n_pinned = 0;
      if (e->cfg.policy_flags & POLICY_NO_LIFECYCLE) {
        a = nb;   // no lifecycle information: nothing is known to be Temporary, everything is admitted
      } else {
        while (a < nb && br[a] != 0) { c.n_pinned += br[a] == 3; ++a; }
      }
      c.n_admissible = a - h;
      e->st.blocks_hashed += nb;
      e->st.hits_hbm += c.n_hit_hbm;
      e->st.hits_host += c.n_hit_host;
      e->st.hits_remote += c.n_hit_remote;
      e->st.misses += nb - h;
      out[i] = CallInfo{nb, h, c.n_hit_hbm, c.n_hit_host, c.n_admissible, 0, c.held, c.n_pinned, c.n_hit_remote};
    }
    return OK;
  }
  // ADMIT: Algorithm 1 with eviction already done by the caller: admit iff a slot is free.
  for (uint32_t i = 0; i < n_ctx; ++i) {
    Ctx &c = e->ctxs[ids[i]];
    uint32_t lim = c.hit_len + c.n_admissible;
    uint32_t b = c.held;
    for (; b < lim; ++b) {
      uint64_t key = c.mat_keys[b];
      Entry *x = find_entry(*e, key);
      if (x) {  // orphan or inserted earlier in this batch: adopt
        x->stamp = e->now;
        x->inflight += 1;
        e->st.adopted++;
      } else if (!e->free_slots[TIER_HBM].empty()) {
        uint32_t slot = *e->free_slots[TIER_HBM].begin();
        e->free_slots[TIER_HBM].erase(e->free_slots[TIER_HBM].begin());
        Entry &n = e->ent[TIER_HBM][slot];
        n.key = key; n.stamp = e->now; n.depth = b; n.inflight = 1; n.floor = 0;
        e->where[key] = {TIER_HBM, slot};
        e->st.inserted++;
      } else {
        break;
      }
    }
    uint32_t adm = b - c.held;
    c.held = b;
    out[i] = CallInfo{(uint32_t)c.mat_keys.size(), c.hit_len, c.n_hit_hbm, c.n_hit_host, c.n_admissible, adm, c.held, c.n_pinned,
                      c.n_hit_remote};
  }
  return OK;
}

int32_t kvto_get_block_map(Engine *e, uint32_t ctx, uint64_t *keys, uint8_t *tier, uint32_t *slot,
                           uint32_t cap, uint32_t *n) {
  if (!e || !n) return E_INVAL;
  Ctx *c = get_ctx(*e, ctx, true);
  if (!c) return E_NOCTX;
  uint32_t nb = (uint32_t)c->mat_keys.size();
  *n = nb;
  if (cap < nb) return E_BUFSZ;
  for (uint32_t b = 0; b < nb; ++b) {
    auto it = e->where.find(c->mat_keys[b]);
    if (keys) keys[b] = c->mat_keys[b];
    if (tier) tier[b] = it == e->where.end() ? 0xFF : (uint8_t)it->second.first;
    if (slot) slot[b] = it == e->where.end() ? 0xFFFFFFFFu : it->second.second;
  }
  return OK;
}

int32_t kvto_get_states(Engine *e, uint32_t tier, uint8_t *state, uint32_t cap) {
  if (!e || !state || tier >= N_TIERS) return E_INVAL;
  if (cap < tier_size(*e, tier)) return E_BUFSZ;
  std::vector<uint8_t> rank[N_TIERS];
  classify(*e, rank);
  if (!rank[tier].empty()) std::memcpy(state, rank[tier].data(), rank[tier].size());
  return OK;
}

// The definition of Section 6.1 written as the literal double loop over (resident block) x (every
// mapping of every context), with block ranks recomputed from token spans per block. Quadratic:
// tiny pools only. Serves as a pin for classify().
int32_t kvto_classify_bruteforce(Engine *e, uint32_t tier, uint8_t *state, uint32_t cap) {
  if (!e || !state || tier >= N_TIERS) return E_INVAL;
  if (cap < tier_size(*e, tier)) return E_BUFSZ;
  for (uint32_t s = 0; s < tier_size(*e, tier); ++s) {
    const Entry &x = e->ent[tier][s];
    if (!x.key) { state[s] = 0xFF; continue; }
    if (x.shadow) { state[s] = 0xFE; continue; }
    int best = x.floor;
    for (const Ctx &c : e->ctxs) {
      if (!c.live) continue;
      std::vector<uint64_t> keys;
      hash_blocks(e->hp, c.mat_tokens.data(), c.mat_tokens.size(), keys);
      for (uint32_t b = 0; b < c.valid_blocks; ++b) {
        if (keys[b] != x.key) continue;
        if (e->cfg.policy_flags & POLICY_ORPHANS_DEAD) {   // reachable: every block of the prefix is resident
          bool reach = true;
          for (uint32_t p = 0; p < b && reach; ++p) reach = e->where.count(keys[p]) != 0;
          if (!reach) continue;
        }
        for (size_t j = 0; j < c.mat_bounds.size(); ++j) {
          uint32_t lo = std::max<uint32_t>(c.mat_bounds[j].first, 16 * b);
          uint32_t hi = std::min<uint32_t>(c.mat_bounds[j].second, 16 * b + 16);
          if (lo < hi) best = std::max(best, msgrank(c.msgs[j].state));
        }
      }
    }
    state[s] = (uint8_t)best;
  }
  return OK;
}

int32_t kvto_select_victims(Engine *e, uint32_t tier, uint32_t n_req, uint32_t flags, uint32_t *slots_out,
                            uint8_t *states_out, uint32_t cap, uint32_t *n_out) {
  if (!e || tier >= N_TIERS || flags > 1 || !n_out || (!slots_out && cap)) return E_INVAL;
  const int max_rank = (flags & 1) ? 3 : 2;   // Pinned KV competes only when the incoming KV is Pinned
  std::vector<uint8_t> rank[N_TIERS];
  classify(*e, rank);
  if (e->cfg.policy_flags & POLICY_NO_LIFECYCLE)   // without lifecycle tracking every resident block is one tier
    for (uint8_t &r : rank[tier]) if (r != 0xFF) r = 1;
  struct Cand { uint32_t slot; uint8_t rank; uint32_t stamp, depth; bool shadow; };
  std::vector<Cand> cands;
  for (uint32_t s = 0; s < tier_size(*e, tier); ++s) {
    const Entry &x = e->ent[tier][s];
    if (!x.key) continue;
    if (x.shadow) { cands.push_back(Cand{s, 0xFE, x.stamp, x.depth, true}); continue; }   // free to drop: first
    if (x.inflight || rank[tier][s] > max_rank) continue;
    // an HBM victim that still has a clean host copy is flagged: moving it out needs no copy
    cands.push_back(Cand{s, (uint8_t)(rank[tier][s] | (x.link >= 0 ? 0x80 : 0)), x.stamp, x.depth, false});
  }
  const bool mru = e->cfg.suspended_order == ORDER_MRU;
  std::stable_sort(cands.begin(), cands.end(), [mru](const Cand &a, const Cand &b) {
    if (a.shadow != b.shadow) return a.shadow;                // host copies of HBM blocks go first
    int ra = a.shadow ? 0 : (a.rank & 0x7F), rb = b.shadow ? 0 : (b.rank & 0x7F);
    if (ra != rb) return ra < rb;                              // Algorithm 1: dead, idle, active, (pinned)
    if (a.stamp != b.stamp) {
      if (ra == 1 && mru && !a.shadow) return a.stamp > b.stamp;   // Section 6.2: most recently suspended first
      return a.stamp < b.stamp;                                // oldest first
    }
    if (a.depth != b.depth) return a.depth > b.depth;          // chain tail before its prefix
    return a.slot < b.slot;
  });
  uint32_t n = std::min<uint32_t>(n_req, (uint32_t)cands.size());
  *n_out = n;
  if (cap < n) return E_BUFSZ;
  for (uint32_t i = 0; i < n; ++i) {
    slots_out[i] = cands[i].slot;
    if (states_out) states_out[i] = cands[i].rank;
  }
  return OK;
}

static int32_t validate_slots(Engine *e, uint32_t tier, const uint32_t *slots, uint32_t n, bool allow_inflight,
                              bool allow_shadow = true) {
  bool bad_range = false, bad_inval = false, bad_state = false;
  std::set<uint32_t> seen;
  for (uint32_t i = 0; i < n; ++i) {
    if (slots[i] >= tier_size(*e, tier)) { bad_range = true; continue; }
    const Entry &x = e->ent[tier][slots[i]];
    if (!x.key || !seen.insert(slots[i]).second || (x.shadow && !allow_shadow)) { bad_inval = true; continue; }
    if (x.inflight && !allow_inflight) bad_state = true;
  }
  if (bad_range) return E_RANGE;
  if (bad_inval) return E_INVAL;
  if (bad_state) return E_STATE;
  return OK;
}

static void move_entry(Engine *e, uint32_t st, uint32_t ss, uint32_t dt, uint32_t ds) {
  copy_payload(*e, st, ss, dt, ds);
  Entry x = e->ent[st][ss];
  e->ent[st][ss] = Entry();
  e->free_slots[st].insert(ss);
  e->free_slots[dt].erase(ds);
  e->ent[dt][ds] = x;
  if (!x.shadow) e->where[x.key] = {dt, ds};
  if (x.link >= 0) e->ent[x.shadow ? TIER_HBM : TIER_HOST][x.link].link = ds;   // the partner follows (compaction)
}

int32_t kvto_offload(Engine *e, const uint32_t *slots, uint32_t n, uint32_t *n_done, uint32_t *n_dropped) {
  if (!e || (!slots && n) || !n_done || !n_dropped) return E_INVAL;
  *n_done = *n_dropped = 0;
  int32_t v = validate_slots(e, TIER_HBM, slots, n, false);
  if (v != OK) return v;
  std::vector<uint8_t> rank[N_TIERS];
  classify(*e, rank);
  const bool knows_dead = !(e->cfg.policy_flags & POLICY_NO_LIFECYCLE);
  // destination slots: the host slots that are free when the call begins, lowest first (slots freed by this
  // call's own drops are not reused within it)
  std::vector<uint32_t> dests(e->free_slots[TIER_HOST].begin(), e->free_slots[TIER_HOST].end());
  size_t next_dest = 0;
  for (uint32_t i = 0; i < n; ++i) {
    uint32_t s = slots[i];
    if (knows_dead && rank[0][s] == 0) {  // reclaim dead KV without a copy
      free_slot(*e, TIER_HBM, s);
      e->st.dropped++;
      (*n_dropped)++;
    } else if (e->ent[TIER_HBM][s].link >= 0) {  // a clean host copy exists: hand the block over, no copy
      Entry x = e->ent[TIER_HBM][s];
      Entry &h = e->ent[TIER_HOST][x.link];
      h.shadow = false; h.link = -1; h.stamp = x.stamp; h.depth = x.depth; h.floor = x.floor; h.inflight = x.inflight;
      e->where[x.key] = {TIER_HOST, (uint32_t)x.link};
      e->ent[TIER_HBM][s] = Entry();
      e->free_slots[TIER_HBM].insert(s);
      e->st.offloaded++;
      e->st.offloaded_clean++;
    } else {
      if (next_dest == dests.size()) return E_NOSPACE;
      uint32_t d = dests[next_dest++];
      move_entry(e, TIER_HBM, s, TIER_HOST, d);
      e->st.offloaded++;
      e->st.bytes_d2h += e->block_bytes;
    }
    (*n_done)++;
  }
  return OK;
}

int32_t kvto_reload(Engine *e, const uint32_t *slots, uint32_t n, uint32_t *n_done) {
  if (!e || (!slots && n) || !n_done) return E_INVAL;
  *n_done = 0;
  int32_t v = validate_slots(e, TIER_HOST, slots, n, true, false);
  if (v != OK) return v;
  for (uint32_t i = 0; i < n; ++i) {
    if (e->free_slots[TIER_HBM].empty()) return E_NOSPACE;
    uint32_t d = *e->free_slots[TIER_HBM].begin();
    if (e->cfg.policy_flags & POLICY_INCLUSIVE) {   // the host slot keeps the bytes as a clean copy
      uint32_t h = slots[i];
      copy_payload(*e, TIER_HOST, h, TIER_HBM, d);
      Entry x = e->ent[TIER_HOST][h];
      x.link = h;
      e->ent[TIER_HBM][d] = x;
      e->free_slots[TIER_HBM].erase(d);
      e->ent[TIER_HOST][h].shadow = true;
      e->ent[TIER_HOST][h].link = d;
      e->ent[TIER_HOST][h].inflight = 0;
      e->where[x.key] = {TIER_HBM, d};
    } else {
      move_entry(e, TIER_HOST, slots[i], TIER_HBM, d);
    }
    e->st.reloaded++;
    e->st.bytes_h2d += e->block_bytes;
    (*n_done)++;
  }
  return OK;
}

// Movement between any two neighbouring levels of the hierarchy (Section 7: HBM, host memory, remote memory), plus
// the direct way up from the remote tier into HBM. Downward (host -> remote) behaves like an offload: dead blocks
// are dropped, live ones go to the destination slots that are free when the call begins, lowest first. Upward
// (remote -> host, remote -> HBM) behaves like a reload: the i-th listed block goes to the i-th lowest free slot;
// blocks in flight may move up (a call fetches its own hits). Clean host copies of HBM blocks cannot be moved.
int32_t kvto_move(Engine *e, uint32_t st, uint32_t dt, const uint32_t *slots, uint32_t n, uint32_t *n_done,
                  uint32_t *n_dropped) {
  if (!e || (!slots && n) || !n_done || !n_dropped) return E_INVAL;
  *n_done = *n_dropped = 0;
  if (st == TIER_HBM && dt == TIER_HOST) return kvto_offload(e, slots, n, n_done, n_dropped);
  if (st == TIER_HOST && dt == TIER_HBM) return kvto_reload(e, slots, n, n_done);
  const bool down = st == TIER_HOST && dt == TIER_REMOTE;
  const bool up = st == TIER_REMOTE && (dt == TIER_HOST || dt == TIER_HBM);
  if (!down && !up) return E_INVAL;
  int32_t v = validate_slots(e, st, slots, n, up, false);
  if (v != OK) return v;
  std::vector<uint8_t> rank[N_TIERS];
  classify(*e, rank);
  const bool knows_dead = !(e->cfg.policy_flags & POLICY_NO_LIFECYCLE);
  // destinations as in kvto_offload: the slots free when the call begins. (Here that is the same set as "free at
  // each step": a drop frees a slot of the source tier only, never one of the destination tier.)
  std::vector<uint32_t> dests(e->free_slots[dt].begin(), e->free_slots[dt].end());
  size_t next_dest = 0;
  for (uint32_t i = 0; i < n; ++i) {
    uint32_t s = slots[i];
    if (down && knows_dead && rank[st][s] == 0) {
      free_slot(*e, st, s);
      e->st.dropped++;
      (*n_dropped)++;
    } else {
      if (next_dest == dests.size()) return E_NOSPACE;
      move_entry(e, st, s, dt, dests[next_dest++]);
      if (down) e->st.demoted++; else e->st.promoted++;
      if (dt == TIER_HBM) e->st.bytes_h2d += e->block_bytes;
    }
    (*n_done)++;
  }
  return OK;
}

// Offload and reload in one call. Both lists are checked against the state the call finds; after that the result is
// by definition that of kvt_offload(out) followed by kvt_reload(in): victims leave first (to the host slots that
// are free when the call begins), the listed host blocks then take the lowest free HBM slots, those the victims
// just left included. (What a device gains from the single call is that the two payload streams can run at the
// same time over a duplex link.)
int32_t kvto_exchange(Engine *e, const uint32_t *out_slots, uint32_t n_out, const uint32_t *in_slots, uint32_t n_in,
                      uint32_t *n_out_done, uint32_t *n_dropped, uint32_t *n_in_done) {
  if (!e || (!out_slots && n_out) || (!in_slots && n_in) || !n_out_done || !n_dropped || !n_in_done) return E_INVAL;
  *n_out_done = *n_dropped = *n_in_done = 0;
  int32_t va = validate_slots(e, TIER_HOST, in_slots, n_in, true, false);
  int32_t vb = validate_slots(e, TIER_HBM, out_slots, n_out, false);
  for (int32_t code : {E_RANGE, E_INVAL, E_STATE})
    if (va == code || vb == code) return code;
  int32_t r_out = kvto_offload(e, out_slots, n_out, n_out_done, n_dropped);
  int32_t r_in = kvto_reload(e, in_slots, n_in, n_in_done);
  return (r_out == E_NOSPACE || r_in == E_NOSPACE) ? E_NOSPACE : OK;
}

int32_t kvto_release(Engine *e, uint32_t tier, const uint32_t *slots, uint32_t n) {
  if (!e || tier >= N_TIERS || (!slots && n)) return E_INVAL;
  int32_t v = validate_slots(e, tier, slots, n, false);
  if (v != OK) return v;
  for (uint32_t i = 0; i < n; ++i) {
    free_slot(*e, tier, slots[i]);
    e->st.dropped++;
  }
  return OK;
}

int32_t kvto_compact(Engine *e, uint32_t tier, uint32_t *n_moved) {
  if (!e || tier >= N_TIERS || !n_moved) return E_INVAL;
  uint32_t n = tier_size(*e, tier);
  uint32_t n_occ = n - (uint32_t)e->free_slots[tier].size();
  std::vector<uint32_t> holes, movers;
  for (uint32_t s = 0; s < n_occ; ++s) if (!e->ent[tier][s].key) holes.push_back(s);
  for (uint32_t s = n_occ; s < n; ++s) if (e->ent[tier][s].key) movers.push_back(s);
  for (size_t i = 0; i < movers.size(); ++i) {
    move_entry(e, tier, movers[i], tier, holes[i]);
    e->st.compacted++;
    e->st.bytes_d2d += e->block_bytes;
  }
  *n_moved = (uint32_t)movers.size();
  return OK;
}

int32_t kvto_copy_blocks(Engine *e, uint32_t st, const uint32_t *src, uint32_t dt, const uint32_t *dst, uint32_t n) {
  if (!e || st >= N_TIERS || dt >= N_TIERS || ((!src || !dst) && n)) return E_INVAL;
  if (!e->cfg.hbm_pool) return E_INVAL;
  for (uint32_t i = 0; i < n; ++i)
    if (src[i] >= tier_size(*e, st) || dst[i] >= tier_size(*e, dt)) return E_RANGE;
  for (uint32_t i = 0; i < n; ++i) copy_payload(*e, st, src[i], dt, dst[i]);
  return OK;
}

int32_t kvto_get_stats(Engine *e, Stats *out) {
  if (!e || !out) return E_INVAL;
  Stats s = e->st;
  s.clock = e->now;
  s.n_contexts = 0;
  for (const Ctx &c : e->ctxs) s.n_contexts += c.live;
  s.occ_hbm = e->cfg.n_hbm_blocks - e->free_slots[0].size();
  s.occ_host = e->cfg.n_host_blocks - e->free_slots[1].size();
  s.occ_remote = e->cfg.n_remote_blocks - e->free_slots[2].size();
  *out = s;
  return OK;
}

int32_t kvto_get_entries(Engine *e, uint32_t tier, uint64_t *keys, uint32_t *stamp, uint32_t *depth,
                         uint32_t *inflight, uint32_t *link, uint32_t cap) {
  if (!e || tier >= N_TIERS) return E_INVAL;
  if (cap < tier_size(*e, tier)) return E_BUFSZ;
  for (uint32_t s = 0; s < tier_size(*e, tier); ++s) {
    const Entry &x = e->ent[tier][s];
    if (keys) keys[s] = x.key;
    if (stamp) stamp[s] = x.stamp;
    if (depth) depth[s] = x.depth;
    if (inflight) inflight[s] = x.inflight;
    if (link) link[s] = x.link >= 0 ? (uint32_t)x.link : 0xFFFFFFFFu;
  }
  return OK;
}

int32_t kvto_debug_load_resident(Engine *e, const uint64_t *keys, const uint8_t *state, const uint32_t *stamp,
                                 const uint32_t *depth, const uint32_t *slot, uint32_t tier, uint32_t n) {
  if (!e || tier >= N_TIERS || ((!keys || !state || !stamp || !depth || !slot) && n)) return E_INVAL;
  std::set<uint64_t> kseen;
  std::set<uint32_t> sseen;
  for (uint32_t i = 0; i < n; ++i) {
    if (keys[i] < 2 || state[i] > 3 || slot[i] >= tier_size(*e, tier)) return E_INVAL;
    if (e->where.count(keys[i]) || e->ent[tier][slot[i]].key) return E_INVAL;
    if (!kseen.insert(keys[i]).second || !sseen.insert(slot[i]).second) return E_INVAL;
  }
  for (uint32_t i = 0; i < n; ++i) {
    Entry &x = e->ent[tier][slot[i]];
    x.key = keys[i]; x.stamp = stamp[i]; x.depth = depth[i]; x.inflight = 0; x.floor = state[i];
    e->free_slots[tier].erase(slot[i]);
    e->where[keys[i]] = {tier, slot[i]};
    if (stamp[i] > e->now) e->now = stamp[i];
  }
  return OK;
}

// ---- all-cores timing helpers --------------------------------------------------------------------------------
// The two embarrassingly parallel stages (block digests, block copies) spread over plain std::threads, for the
// benchmark's "all host cores" figures. They are not part of the engine above and nothing else calls them.
int32_t kvto_par_digests(const uint32_t *tokens, uint64_t n_tokens, uint64_t seed, uint64_t *digests, uint32_t n_threads) {
  if ((!tokens || !digests) && n_tokens >= 16) return E_INVAL;
  if (!n_threads) return E_INVAL;
  const HashParams hp = make_params(seed);
  const uint64_t nb = n_tokens / 16;
  std::vector<std::thread> th;
  for (uint32_t t = 0; t < n_threads; ++t)
    th.emplace_back([=, &hp]() {
      for (uint64_t b = nb * t / n_threads; b < nb * (t + 1) / n_threads; ++b) {
        uint64_t sum = 0;
        for (int k = 0; k < 16; ++k) sum += ((uint64_t)tokens[16 * b + k] + 1ull) * hp.K[k];
        digests[b] = mix64(sum);
      }
    });
  for (auto &x : th) x.join();
  return OK;
}

int32_t kvto_par_copy_blocks(uint8_t *dst, const uint8_t *src, uint64_t block_bytes, const uint32_t *src_ids,
                             const uint32_t *dst_ids, uint32_t n, uint32_t n_threads) {
  if (!dst || !src || !src_ids || !dst_ids || !n_threads) return E_INVAL;
  std::vector<std::thread> th;
  for (uint32_t t = 0; t < n_threads; ++t)
    th.emplace_back([=]() {
      for (uint64_t i = (uint64_t)n * t / n_threads; i < (uint64_t)n * (t + 1) / n_threads; ++i)
        std::memcpy(dst + (uint64_t)dst_ids[i] * block_bytes, src + (uint64_t)src_ids[i] * block_bytes, block_bytes);
    });
  for (auto &x : th) x.join();
  return OK;
}

}  // extern "C"
