// kvt_engine.cu — host control plane and C ABI of libkvt.so (see include/kvt.h for the contract).
//
// The host side keeps only what a data-parallel kernel cannot: per-context message lists (lengths
// and message-level states, Section 5.2), the materialised message bounds (Section 5.1), range
// allocators for the caller-provided arenas, counts of free slots, and the logical clock. Token
// values, block keys, the block table, per-block metadata and payloads live on the device and are
// only touched by the kernels in kvt_kernels.cuh. There is no CPU fallback for any stage.
#include "kvt_kernels.cuh"

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <string>
#include <vector>

#include "../../include/kvt.h"

using namespace kvt;

namespace {

// Threads per block of the element-wise kernels. The checked build (-DKVT_DEBUG) runs every launch in another
// shape (small blocks, a handful of mover CTAs, no CUDA graph): results do not depend on the shape, and a kernel
// that secretly relied on it shows up as a difference from the CPU reference in the tests.
#ifdef KVT_DEBUG
constexpr u32 TPB = 64;
constexpr bool CHECKED_BUILD = true;
#else
constexpr u32 TPB = 256;
constexpr bool CHECKED_BUILD = false;
#endif

constexpr u32 MS_ACTIVE = 0, MS_SUSPENDED = 1, MS_EXPIRED = 2, MS_TEMPORARY = 3, MS_PINNED = 4;
// Priority of a message state in the block aggregate: Algorithm 1's release order.
inline u8 msg_rank(u8 s) { return s == MS_PINNED ? 3 : (s == MS_ACTIVE ? 2 : (s == MS_SUSPENDED ? 1 : 0)); }

inline u64 round_up(u64 x, u64 a) { return (x + a - 1) / a * a; }
inline u32 cdiv(u64 a, u64 b) { return (u32)((a + b - 1) / b); }
inline u32 bit_length(u32 x) { u32 n = 0; while (x) { ++n; x >>= 1; } return n ? n : 1; }

// First-fit range allocator over a caller-provided arena (units: elements).
struct RangeAlloc {
  std::map<u64, u64> free_;
  u64 align = 1;
  void init(u64 total, u64 a) { free_.clear(); align = a; if (total) free_[0] = total / a * a; }
  bool alloc(u64 n, u64 *off) {
    n = round_up(std::max<u64>(n, 1), align);
    for (auto it = free_.begin(); it != free_.end(); ++it) {
      if (it->second >= n) {
        *off = it->first;
        u64 rest = it->second - n, ro = it->first + n;
        free_.erase(it);
        if (rest) free_[ro] = rest;
        return true;
      }
    }
    return false;
  }
  void release(u64 off, u64 n) {
    n = round_up(std::max<u64>(n, 1), align);
    auto nx = free_.lower_bound(off);
    if (nx != free_.end() && off + n == nx->first) { n += nx->second; nx = free_.erase(nx); }
    if (nx != free_.begin()) {
      auto pv = std::prev(nx);
      if (pv->first + pv->second == off) { pv->second += n; return; }
    }
    free_[off] = n;
  }
};

struct Msg { u32 len; u8 state; };
// A key list in the key arena: keycap keys followed by one chain carry per CHUNK keys (kept so that the next
// call can resume hashing at a chunk boundary instead of block 0).
struct KeySeg { u64 off = 0, cap = 0, keycap = 0; u32 refs = 0; };

// What the per-block mapping counts currently contain for one context: the key list, the mapped prefix length and
// the message table (slice of the device message arrays) it was accounted with. Holds a reference on the key segment.
struct Snap { int keyseg = -1; u32 valid = 0; u64 tbl_off = 0; u32 tbl_n = 0; };

struct Ctx {
  bool live = false, one_off = false, in_flight = false;
  bool map_dirty = false;    // messages, mapped prefix or key list changed since `synced` was taken
  Snap synced;
  bool terminated = false;   // ended but kept: it still has Pinned messages
  std::vector<Msg> msgs;
  std::vector<std::pair<u32, u32>> mat_bounds;  // bounds of the leading messages still valid in the materialised layout
  u32 mat_blocks = 0;      // blocks of the materialised token sequence (keys in the key segment)
  u32 valid_blocks = 0, held = 0, hit_len = 0, n_hit_hbm = 0, n_hit_host = 0, n_hit_remote = 0, n_admissible = 0, n_pinned = 0;
  u64 tok_off = 0, tok_cap = 0, tok_len = 0;   // device token buffer = concatenation of the current messages
  int keyseg = -1;
};

struct DevLayout {
  u64 tab, e_key, e_stamp, e_depth, e_infl, e_cnt, e_tslot, e_mark, e_link, e_floor, cnt_chk, fresh, keys, status;
  u64 s0, s1, s2, s3, ids, ids2, pair_src, pair_dst, pair_src2, pair_dst2, freelist, freelist2, tiles, agg, carry, cflags, desc, ctxres;
  u64 m_start, m_end, m_rank, keyA, keyB, valA, valB, rcounts, sel_cta, sel_args, slot_key, sel_hist, sel_state, out_slots, out_states, map_tier, map_slot;
  u64 total;
  u64 LB, Nt, N;
};

DevLayout make_layout(const kvt_config &c) {
  DevLayout L{};
  u64 N = (u64)c.n_hbm_blocks + c.n_host_blocks + c.n_remote_blocks;
  u64 Nt = std::max(std::max(c.n_hbm_blocks, c.n_host_blocks), c.n_remote_blocks);
  u64 B = c.max_batch_blocks, LB = std::max<u64>(B, Nt), C = c.max_contexts, Mm = c.max_messages;
  L.LB = LB; L.Nt = Nt; L.N = N;
  u64 off = 0;
  auto take = [&](u64 bytes) { u64 o = off; off = round_up(off + bytes, 256); return o; };
  L.tab = take((u64)c.table_capacity * 16);
  L.e_key = take(N * 8); L.e_stamp = take(N * 4); L.e_depth = take(N * 4); L.e_infl = take(N * 4);
  L.e_cnt = take(N * 8); L.e_tslot = take(N * 4); L.e_mark = take(N * 4); L.e_link = take(N * 4); L.e_floor = take(N);
  L.cnt_chk = take(N * 8);   // the counts of a full recomputation, for the cross-check mode
  L.fresh = take(N * 4);     // entries inserted since the counts were last brought up to date
  L.keys = take((c.max_key_blocks + c.max_key_blocks / CHUNK + 64ull * c.max_contexts) * 8);   // keys + per-chunk carries
  // status words, per-context results and call descriptors sit in one stretch, on the device and in the pinned
  // staging area alike, so that a LOOKUP call uploads all three with one copy and reads two of them back with one
  L.status = take(ST_WORDS * 4);
  L.ctxres = take(C * 20);   // per context: hit_len, hits per tier (3), admission stop
  L.desc = take(C * 256 + 2 * (B / CHUNK + C + 1) * 4);  // per-context descriptors, then the chunk -> context maps of a LOOKUP batch
  L.s0 = take(LB * 4); L.s1 = take(LB * 4); L.s2 = take(LB * 4); L.s3 = take(LB * 4);
  L.ids = take(LB * 4); L.ids2 = take(LB * 4); L.pair_src = take(LB * 4); L.pair_dst = take(LB * 4);
  L.freelist = take(LB * 4); L.freelist2 = take(LB * 4); L.pair_src2 = take(LB * 4); L.pair_dst2 = take(LB * 4);
  L.tiles = take((std::max(LB, N) / SCAN_TILE + 2) * 4);
  u64 n_chunks = B / CHUNK + C + 1;
  L.agg = take(n_chunks * 8); L.carry = take(n_chunks * 8);   // per-chunk aggregates / chain values of a LOOKUP batch
  L.cflags = take((n_chunks + 1) * 4);                         // per-chunk publication flags + the ticket word
  L.m_start = take(2 * Mm * 4); L.m_end = take(2 * Mm * 4); L.m_rank = take(2 * Mm);   // accounted-for tables + the new ones of a pass
  L.keyA = take(Nt * 8); L.keyB = take(Nt * 8); L.valA = take(Nt * 4); L.valB = take(Nt * 4);
  L.rcounts = take(((u64)RADIX_BINS * (Nt / SORT_TILE + 1) + RADIX_BINS) * 4);
  L.sel_cta = take((Nt / SEL_TILE + 2) * 4);
  L.sel_args = take(sizeof(SelArgs));
  L.slot_key = take(Nt * 8);
  L.sel_hist = take((u64)SEL_MAX_LEVELS * SEL_BINS * 4);
  L.sel_state = take((SEL_MAX_LEVELS + 1) * sizeof(SelState));
  L.out_slots = take(Nt * 4); L.out_states = take(Nt);
  L.map_tier = take(B); L.map_slot = take(B * 4);
  L.total = off;
  return L;
}

}  // namespace

struct kvt_engine {
  kvt_config cfg;
  DevLayout L;
  u8 *meta = nullptr;
  u32 *d_tokens = nullptr;
  Table tab; Entries ent;
  u64 *d_keys; u32 *d_status;
  u64 h0;
  u64 chunk_bytes, n_chunks, block_bytes;
  bool metadata_only;
  int sm_count = 148;
  // host state
  std::vector<Ctx> ctxs;
  std::vector<KeySeg> segs;
  std::vector<int> free_segs;
  RangeAlloc tok_alloc, key_alloc;
  u32 now = 0, max_depth = 0;
  u32 occ[3] = {0, 0, 0};
  u32 tombs = 0;
  bool dirty = true;          // something below is pending: the counts are not up to date
  bool full_dirty = true;     // the counts must be recomputed from scratch (start; debug loads; after an arena ran out)
  std::vector<Snap> zombies;  // what is still accounted for contexts that have ended
  u32 n_fresh = 0;            // entries in the device list L.fresh
  RangeAlloc tbl_alloc;       // slices of the device message arrays
  u32 classify_mode = 0;      // 0 event-driven, 1 full recomputation every time, 2 event-driven + cross-check
  kvt_stats st{};
  std::string err;
  // pinned host staging
  u8 *stage = nullptr;
  u32 *h_status; u8 *h_desc; u32 *h_ctxres; u32 *h_mstart, *h_mend; u8 *h_mrank; u32 *h_ids, *h_ids2; u8 *h_out;   // h_out: results staged for the caller (block maps, victim lists)
  cudaEvent_t ev_upload = nullptr;
  bool upload_pending = false;
  // optional timing of the mover kernel (kvt_set_profiling)
  bool profiling = false, mover_timed = false;
  // CUDA graph of the kernel sequence of kvt_select_victims, one per tier
  struct SelGraph { cudaGraphExec_t exec = nullptr; };
  std::map<u64, SelGraph> sel_graph[3];    // keyed by (level count, pass count, sort tiles)
  cudaStream_t capture_stream = nullptr;   // only ever used for stream capture, never executes work
  bool use_graphs = true;
  SelArgs *h_sel = nullptr;                // pinned staging of the selection's argument record
  u32 mover_variant = 0;   // 0 auto, 1 CTA per chunk, 2 warp per 4 KiB tile, 3 TMA ring, 4 copy engines through the staging ring
  // Staging ring for moves between device memory and a pool in host memory: the payload is gathered into (scattered
  // from) contiguous device memory by the mover kernel and crosses the link as large copy-engine transfers on the
  // library's own two copy streams (one per direction, so an exchange drives the link in both directions).
  static constexpr int N_STAGES = 4;
  struct Staging {
    u8 *buf = nullptr; u32 blocks_per_stage = 0; bool ok = false;
    cudaStream_t cs[2] = {nullptr, nullptr};                 // [0] device -> host, [1] host -> device
    cudaEvent_t ready[2][N_STAGES] = {}, free_[2][N_STAGES] = {}, begin = nullptr;
  } stg;
  u32 mover_max_ctas = 0;  // caller's upper bound on the mover's grid (0: automatic)
  bool tier_in_host_mem[3] = {false, false, false};   // pool is host memory: moves to / from it are bound by the host link
  // Grid of a mover launch. Inside the device: 8 CTAs of 256 threads per SM. A move that crosses the host link
  // is bound by the link: 128 warps keep it full (measured), and a GEMM on another stream loses every SM a mover
  // CTA sits on, so those warps are packed into 4 CTAs of 1024 threads (8 for an exchange, which
  // drives both directions).
  u32 mover_grid(u64 want, u32 link_dirs = 0) const {
    u64 cap = mover_max_ctas ? mover_max_ctas : CHECKED_BUILD ? 5 : link_dirs == 1 ? 4 : link_dirs == 2 ? 8 : (u64)sm_count * 8;
    return (u32)std::max<u64>(1, std::min(want, cap));
  }
  u32 link_dirs(u32 st, u32 dt) const { return (tier_in_host_mem[st] || tier_in_host_mem[dt]) ? 1u : 0u; }
  // L2 residency of the block table and the hot per-entry arrays (key, stamp, depth, in-flight, counts): the kernels
  // that probe them are launched with an access-policy window over that range, so the lines they touch stay in the
  // persisting part of L2 while KV payload and token streams pass through the rest
  cudaAccessPolicyWindow l2_win{};
  bool l2_on = false;
  u32 copy_delay_ns = 0;   // test hook: the control-record copy kernels start their copy this much later
  bool overlap_launches = !CHECKED_BUILD;   // dependent launches inside one call (digest -> finish -> lock)
  u32 lookup_variant = 0;  // 0 / 1 digest / carry / finish kernels, 2 single-pass hash + probe kernel
  u32 wait_limit = 1u << 18;   // polls a chunk of the single-pass kernel spends on its predecessors before it gives up
  bool tma_attr_set = false;
  cudaEvent_t ev_m0 = nullptr, ev_m1 = nullptr, ev_h0 = nullptr, ev_h1 = nullptr, ev_c0 = nullptr, ev_c1 = nullptr;
  bool classify_timed = false; u64 classify_pending_items = 0;   // a timed classification whose events have not been read yet

  template <class T> T *dp(u64 off) const { return reinterpret_cast<T *>(meta + off); }
  u32 tier_slots(u32 t) const { return t == KVT_TIER_HBM ? cfg.n_hbm_blocks : t == KVT_TIER_HOST ? cfg.n_host_blocks : cfg.n_remote_blocks; }
  u32 tier_e0(u32 t) const { return t == KVT_TIER_HBM ? 0 : t == KVT_TIER_HOST ? cfg.n_hbm_blocks : cfg.n_hbm_blocks + cfg.n_host_blocks; }
};

namespace {

#define CU(call)                                                                                   \
  do {                                                                                             \
    cudaError_t _e = (call);                                                                       \
    if (_e != cudaSuccess) {                                                                       \
      e->err = std::string(#call) + ": " + cudaGetErrorString(_e);                                 \
      return KVT_E_CUDA;                                                                           \
    }                                                                                              \
  } while (0)

// every kernel launch of the library goes through this macro, which also counts it
#define KL(kern, grid, block, stream, ...)                     \
  do {                                                         \
    kern<<<(grid), (block), 0, (stream)>>>(__VA_ARGS__);       \
    e->st.kernel_launches++;                                   \
  } while (0)

template <typename... Exp, typename... Act>
void launch_attr(kvt_engine *e, bool window, bool after_kernel, void (*kern)(Exp...), u32 grid, u32 block, cudaStream_t s,
                 Act &&...args);
// Launch of a kernel that works on the block table / per-entry metadata: carries the L2 access-policy window.
// after_kernel: the launch directly follows, in the same stream, a kernel that releases its dependents early; this
// kernel's CTAs may then take the SM slots the tail of that kernel leaves free and wait (dep_wait() in the kernel)
// for its results there, instead of starting after the last CTA has drained.
template <typename... Exp, typename... Act>
void launch_meta(kvt_engine *e, bool after_kernel, void (*kern)(Exp...), u32 grid, u32 block, cudaStream_t s, Act &&...args) {
  launch_attr(e, true, after_kernel, kern, grid, block, s, std::forward<Act>(args)...);
  e->st.kernel_launches++;
}
template <typename... Exp, typename... Act>
void launch_attr(kvt_engine *e, bool window, bool after_kernel, void (*kern)(Exp...), u32 grid, u32 block, cudaStream_t s,
                 Act &&...args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(block); cfg.stream = s;
  cudaLaunchAttribute at[2];
  u32 n = 0;
  if (window && e->l2_on) {
    at[n].id = cudaLaunchAttributeAccessPolicyWindow;
    at[n].val.accessPolicyWindow = e->l2_win;
    ++n;
  }
  if (after_kernel && e->overlap_launches) {
    at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = at; cfg.numAttrs = n;
  cudaLaunchKernelEx(&cfg, kern, std::forward<Act>(args)...);
}
#define KLM(kern, grid, block, stream, ...) launch_meta(e, false, kern, (grid), (block), (stream), __VA_ARGS__)
#define KLD(kern, grid, block, stream, ...) launch_meta(e, true, kern, (grid), (block), (stream), __VA_ARGS__)

int32_t fail(kvt_engine *e, int32_t code, const char *msg) { e->err = msg; return code; }

// Per-kernel timing for development builds (-DKVT_TRACE): an event after every marked launch, the gaps printed to
// stderr once the call has synchronised. Compiles to nothing otherwise.
#ifdef KVT_TRACE
struct Trace { cudaEvent_t ev[64]; const char *name[64]; int n = 0; bool init = false; };
static Trace g_trace;
static void trace_mark(cudaStream_t s, const char *name) {
  Trace &t = g_trace;
  if (!t.init) { for (auto &x : t.ev) cudaEventCreate(&x); t.init = true; }
  if (t.n < 64) { t.name[t.n] = name; cudaEventRecord(t.ev[t.n++], s); }
}
static void trace_dump(const char *what) {
  Trace &t = g_trace;
  if (t.n > 1 && getenv("KVT_TRACE")) {
    fprintf(stderr, "[trace] %s:", what);
    for (int i = 1; i < t.n; ++i) { float ms = 0; cudaEventElapsedTime(&ms, t.ev[i - 1], t.ev[i]); fprintf(stderr, " %s %.1f", t.name[i], ms * 1e3f); }
    float tot = 0; cudaEventElapsedTime(&tot, t.ev[0], t.ev[t.n - 1]);
    fprintf(stderr, " | total %.1f us\n", tot * 1e3f);
  }
  t.n = 0;
}
#define TRACE(s, name) trace_mark(s, name)
#define TRACE_DUMP(what) trace_dump(what)
#else
#define TRACE(s, name) do {} while (0)
#define TRACE_DUMP(what) do {} while (0)
#endif

int32_t launch_ok(kvt_engine *e) {
  cudaError_t x = cudaGetLastError();
  if (x != cudaSuccess) { e->err = std::string("kernel launch: ") + cudaGetErrorString(x); return KVT_E_CUDA; }
  return KVT_OK;
}
#define LAUNCH_CHECK() do { int32_t _r = launch_ok(e); if (_r) return _r; } while (0)

// Staging buffers are reused by every call: wait until the previous upload has been consumed.
int32_t stage_acquire(kvt_engine *e) {
  if (e->upload_pending) { CU(cudaEventSynchronize(e->ev_upload)); e->upload_pending = false; }
  return KVT_OK;
}
int32_t stage_release(kvt_engine *e, cudaStream_t s) {
  CU(cudaEventRecord(e->ev_upload, s));
  e->upload_pending = true;
  return KVT_OK;
}

// Control records between the pinned staging area and device memory, carried by one small kernel instead of one
// copy-engine transfer each (a transfer of a few KB costs 8-11 us of stream time, the kernel 3-5 us for all of them).
// Host-side pointers must lie in the staging area; a pending list is sent with flush().
struct SegCopy {
  kvt_engine *e; cudaStream_t s; CopySegs c{}; bool after_kernel;
  SegCopy(kvt_engine *e_, cudaStream_t s_, bool after_kernel_ = false) : e(e_), s(s_), after_kernel(after_kernel_) { c.n = 0; }
  void add(void *dst, const void *src, u64 bytes) {
    if (!bytes) return;
    if (c.n == 6) flush();
    c.src[c.n] = src; c.dst[c.n] = dst; c.bytes[c.n] = (u32)bytes; ++c.n;
  }
  void flush() {
    if (!c.n) return;
    u64 most = 0;
    for (u32 k = 0; k < c.n; ++k) most = std::max<u64>(most, c.bytes[k]);
    launch_attr(e, false, after_kernel, k_copy_segs, (u32)std::min<u64>(std::max<u64>(cdiv(most / 16, 256), 1), 64), 256u, s, c, e->copy_delay_ns);
    e->st.kernel_launches++;
    c.n = 0; after_kernel = true;
  }
};

int32_t status_zero(kvt_engine *e, cudaStream_t s) {
  CU(cudaMemsetAsync(e->d_status, 0, ST_WORDS * 4, s));
  return KVT_OK;
}
// Copies the status block to the host and waits for the stream.
int32_t status_fetch(kvt_engine *e, cudaStream_t s) {
  CU(cudaMemcpyAsync(e->h_status, e->d_status, ST_WORDS * 4, cudaMemcpyDeviceToHost, s));
  CU(cudaStreamSynchronize(s));
  return KVT_OK;
}
int32_t status_code(kvt_engine *e) {
  u32 b = e->h_status[ST_ERR];
  if (!b) return KVT_OK;
  if (b & DERR_WAIT) return fail(e, KVT_E_DEVICE, "a chunk's wait for its predecessor ran out");
  if (b & (DERR_PROBE | DERR_CORRUPT)) return fail(e, KVT_E_DEVICE, b & DERR_PROBE ? "table probe cap exceeded" : "corrupt metadata");
  if (b & DERR_RANGE) return fail(e, KVT_E_RANGE, "slot id out of range");
  if (b & DERR_INVAL) return fail(e, KVT_E_INVAL, "slot empty, repeated, or key already resident");
  return fail(e, KVT_E_STATE, "block is in flight");
}

Ctx *get_ctx(kvt_engine *e, u32 id, bool allow_terminated = false) {
  if (id >= e->ctxs.size() || !e->ctxs[id].live) return nullptr;
  if (e->ctxs[id].terminated && !allow_terminated) return nullptr;
  return &e->ctxs[id];
}

void seg_deref(kvt_engine *e, int id) {
  if (id < 0) return;
  KeySeg &s = e->segs[id];
  if (--s.refs == 0) { e->key_alloc.release(s.off, s.cap); e->free_segs.push_back(id); }
}
int seg_new(kvt_engine *e, u64 n) {
  u64 keycap = round_up(std::max<u64>(n, 1), 32), total = keycap + cdiv(keycap, (u64)CHUNK) + 1, off;   // one carry per chunk (the last may be partial) + the resume point
  if (!e->key_alloc.alloc(total, &off)) return -1;
  int id;
  if (!e->free_segs.empty()) { id = e->free_segs.back(); e->free_segs.pop_back(); }
  else { id = (int)e->segs.size(); e->segs.emplace_back(); }
  e->segs[id] = KeySeg{off, round_up(total, e->key_alloc.align), keycap, 1};
  return id;
}

// ---- ordered compaction helper -----------------------------------------------------------------------
template <class Pred, class Emit>
int32_t compact_indices(kvt_engine *e, cudaStream_t s, Pred pred, Emit emit, u32 n, int total_word) {
  u32 *tiles = e->dp<u32>(e->L.tiles);
  u32 nt = cdiv(n, SCAN_TILE);
  if (nt == 0) { CU(cudaMemsetAsync(e->d_status + total_word, 0, 4, s)); return KVT_OK; }
  KL(k_tile_count, nt, SCAN_TILE, s, pred, n, tiles);
  KL(k_scan_tiles, 1, 1024, s, tiles, nt, e->d_status + total_word);
  KL(k_tile_scatter, nt, SCAN_TILE, s, pred, emit, n, tiles);
  LAUNCH_CHECK();
  return KVT_OK;
}

int32_t table_rebuild(kvt_engine *e, cudaStream_t s) {
  KL(k_table_clear, cdiv((u64)e->tab.mask + 1, TPB), TPB, s, e->tab);
  KL(k_table_reinsert, cdiv(e->ent.n_total, TPB), TPB, s, e->tab, e->ent, e->d_status);
  LAUNCH_CHECK();
  e->tombs = 0;
  e->st.table_rebuilds++;
  return KVT_OK;
}

int32_t maybe_rebuild(kvt_engine *e, cudaStream_t s) {
  if ((u64)e->tombs * 8 > (u64)e->tab.mask + 1) return table_rebuild(e, s);
  return KVT_OK;
}

PoolView pool_view(kvt_engine *e, u32 tier) {
  PoolView v;
  if (tier == KVT_TIER_HBM) {
    v.base = (u8 *)e->cfg.hbm_pool;
    v.n_slots = e->cfg.n_hbm_blocks;
    if (e->cfg.pool_layout == KVT_LAYOUT_LAYER_MAJOR) { v.slot_stride = e->chunk_bytes; v.chunk_stride = e->chunk_bytes * e->cfg.n_hbm_blocks; }
    else { v.slot_stride = e->block_bytes; v.chunk_stride = e->chunk_bytes; }
  } else {
    v.base = (u8 *)(tier == KVT_TIER_HOST ? e->cfg.host_pool : e->cfg.remote_pool);
    v.n_slots = e->tier_slots(tier);
    v.slot_stride = e->block_bytes; v.chunk_stride = e->chunk_bytes;
  }
  return v;
}

// View of one stage of the staging ring as a block-major pool of `blocks` slots.
PoolView stage_view(kvt_engine *e, int dir, int stage, u32 blocks) {
  PoolView v;
  v.base = e->stg.buf + ((u64)dir * kvt_engine::N_STAGES + stage) * e->stg.blocks_per_stage * e->block_bytes;
  v.n_slots = blocks; v.slot_stride = e->block_bytes; v.chunk_stride = e->chunk_bytes;
  return v;
}

int32_t launch_mover_views(kvt_engine *e, cudaStream_t s, const PoolView &sv, const u32 *src, const PoolView &dv, const u32 *dst,
                           u32 n_max, const u32 *n_dev, u32 ld, bool timed);

int32_t launch_mover(kvt_engine *e, cudaStream_t s, u32 st, const u32 *src, u32 dt, const u32 *dst, u32 n_max,
                     const u32 *n_dev) {
  if (e->metadata_only || n_max == 0) return KVT_OK;
  return launch_mover_views(e, s, pool_view(e, st), src, pool_view(e, dt), dst, n_max, n_dev, e->link_dirs(st, dt),
                            e->profiling && n_dev != nullptr);   // only the calls that synchronise afterwards are timed
}

int32_t launch_mover_views(kvt_engine *e, cudaStream_t s, const PoolView &sv, const u32 *src, const PoolView &dv, const u32 *dst,
                           u32 n_max, const u32 *n_dev, u32 ld, bool timed) {
  MoveArgs a;
  a.src = sv; a.dst = dv;
  a.src_ids = src; a.dst_ids = dst; a.n_pairs = n_max; a.n_pairs_dev = n_dev;
  a.n_chunks = (u32)e->n_chunks; a.chunk_bytes = (u32)e->chunk_bytes; a.status = e->d_status;
  u64 items = (u64)n_max * e->n_chunks;
  u32 grid = e->mover_grid(items, ld) * (ld && !e->mover_max_ctas ? 4 : 1);   // 256-thread CTAs: four for one of 1024
  if (timed) CU(cudaEventRecord(e->ev_m0, s));
  // a warp per 4 KiB tile keeps 8 loads per lane in flight whatever the chunk size (measured faster for
  // 4 KiB and 32 KiB chunks alike); chunks that are not a multiple of 4 KiB take the CTA-per-chunk kernel
  const bool tiles_ok = e->chunk_bytes % 4096 == 0;
  const bool use_tiles = e->mover_variant != 1;
  if (e->mover_variant == 3 && e->chunk_bytes % 16 == 0 && src && dst) {   // TMA ring (experimental variant)
    u32 tile = (u32)(e->chunk_bytes <= 16384 ? e->chunk_bytes : (e->chunk_bytes % 16384 == 0 ? 16384 : 0));
    if (tile == 0 || tile > 49152) return fail(e, KVT_E_INVAL, "chunk size not supported by the TMA mover");
    u32 tpc = (u32)(e->chunk_bytes / tile);
    u64 titems = items * tpc;
    size_t smem = (size_t)TMA_STAGES * tile;
    if (!e->tma_attr_set) {
      CU(cudaFuncSetAttribute(k_move_tma, cudaFuncAttributeMaxDynamicSharedMemorySize, 196608));
      e->tma_attr_set = true;
    }
    u32 per_sm = (u32)std::max<size_t>(1, std::min<size_t>(8, (200 * 1024) / (smem + 1024)));
    u32 tgrid = (u32)std::min<u64>(titems, (u64)e->sm_count * per_sm);
    tgrid = std::min(tgrid, e->mover_grid(titems, ld) * (ld && !e->mover_max_ctas ? 8 : 1));   // one warp per CTA here
    k_move_tma<<<tgrid, 32, smem, s>>>(a, tile, tpc);
    e->st.kernel_launches++;
  } else if (use_tiles && tiles_ok) {
    u32 tpc = (u32)(e->chunk_bytes / 4096);
    u64 titems = items * tpc;
    if (ld) {   // link-bound: few, large CTAs (see mover_grid)
      u32 tgrid = e->mover_grid((titems + 31) / 32, ld);
      KL((k_move_tiles<8, 1024>), tgrid, 1024, s, a, tpc);
    } else {
      u32 tgrid = e->mover_grid((titems + 7) / 8, ld);
      KL(k_move_tiles<8>, tgrid, 256, s, a, tpc);
    }
  } else {
    KL(k_move_blocks<4>, grid, 256, s, a);
  }
  if (timed) { CU(cudaEventRecord(e->ev_m1, s)); e->mover_timed = true; }
  LAUNCH_CHECK();
  return KVT_OK;
}

// Whether a move of n blocks between these tiers goes through the staging ring: a staging buffer is configured,
// exactly one side is a pool in host memory, and the blocks are large enough for one copy-engine transfer each.
bool staged_applies(const kvt_engine *e, u32 st, u32 dt) {
  if (!e->stg.ok || e->metadata_only) return false;
  if (e->tier_in_host_mem[st] == e->tier_in_host_mem[dt]) return false;
  if (e->mover_variant != 0 && e->mover_variant != 4) return false;      // a kernel variant was asked for
  return e->mover_variant == 4 || e->block_bytes >= (512u << 10);
}

// Moves n blocks src_tier[h_src[i]] -> dst_tier[h_dst[i]] through the staging ring; h_src / h_dst are the planned
// pairs on the host. The blocks travel in the order of their slots in the host-memory pool, whatever the order of
// the list (the copies are independent of each other), so that every stretch of consecutive host slots is one
// copy-engine transfer. dir 0: device -> host (gather into a stage on `s`, then transfers on the copy stream);
// dir 1: host -> device (transfers into a stage on the copy stream, then scatter on `s`). When this returns, `s`
// waits for everything the copy stream still has to do.
int32_t staged_move(kvt_engine *e, cudaStream_t s, u32 st, const u32 *h_src, u32 dt, const u32 *h_dst, u32 n) {
  if (!n) return KVT_OK;
  const int dir = e->tier_in_host_mem[st] ? 1 : 0;
  kvt_engine::Staging &g = e->stg;
  const u32 SB = g.blocks_per_stage;
  const u64 BB = e->block_bytes;
  u8 *host_pool = (u8 *)(dir ? (st == KVT_TIER_HOST ? e->cfg.host_pool : e->cfg.remote_pool)
                             : (dt == KVT_TIER_HOST ? e->cfg.host_pool : e->cfg.remote_pool));
  const u32 *h_host = dir ? h_src : h_dst, *h_dev = dir ? h_dst : h_src;   // slots of the host-memory pool / of the device pool
  const u32 n_host_slots = e->tier_slots(dir ? st : dt);
  for (u32 i = 0; i < n; ++i) if (h_host[i] >= n_host_slots) return fail(e, KVT_E_RANGE, "slot id out of range");
  std::vector<u32> order(n), host_sorted(n);
  for (u32 i = 0; i < n; ++i) order[i] = i;
  std::sort(order.begin(), order.end(), [&](u32 x, u32 y) { return h_host[x] < h_host[y]; });
  int32_t r = stage_acquire(e);
  if (r) return r;
  u32 *h_ids = e->h_ids2, *d_ids = e->dp<u32>(e->L.ids2);    // device-pool slots in travelling order
  for (u32 p = 0; p < n; ++p) { h_ids[p] = h_dev[order[p]]; host_sorted[p] = h_host[order[p]]; }
  CU(cudaMemcpyAsync(d_ids, h_ids, n * 4ull, cudaMemcpyHostToDevice, s));
  r = stage_release(e, s);   // the next call that stages ids waits for this upload
  if (r) return r;
  const bool timed = e->profiling;
  if (timed) CU(cudaEventRecord(e->ev_m0, s));
  if (dir == 1) {   // the host pool holds what earlier work on `s` put there
    CU(cudaEventRecord(g.begin, s));
    CU(cudaStreamWaitEvent(g.cs[1], g.begin, 0));
  }
  const u32 n_batches = cdiv(n, SB);
  for (u32 k = 0; k < n_batches; ++k) {
    const int sg = (int)(k % kvt_engine::N_STAGES);
    const u32 b0 = k * SB, nb = std::min(SB, n - b0);
    u8 *stage = stage_view(e, dir, sg, nb).base;
    auto transfers = [&]() -> int32_t {
      for (u32 p = 0; p < nb;) {
        u32 run = 1;
        while (p + run < nb && host_sorted[b0 + p + run] == host_sorted[b0 + p] + run) ++run;
        u8 *hp = host_pool + (u64)host_sorted[b0 + p] * BB, *sp = stage + (u64)p * BB;
        if (dir == 0) CU(cudaMemcpyAsync(hp, sp, run * BB, cudaMemcpyDeviceToHost, g.cs[0]));
        else CU(cudaMemcpyAsync(sp, hp, run * BB, cudaMemcpyHostToDevice, g.cs[1]));
        p += run;
      }
      return KVT_OK;
    };
    if (dir == 0) {
      if (k >= (u32)kvt_engine::N_STAGES) CU(cudaStreamWaitEvent(s, g.free_[0][sg], 0));   // the stage's transfers are done
      r = launch_mover_views(e, s, pool_view(e, st), d_ids + b0, stage_view(e, 0, sg, nb), nullptr, nb, nullptr, 0, false);
      if (r) return r;
      CU(cudaEventRecord(g.ready[0][sg], s));
      CU(cudaStreamWaitEvent(g.cs[0], g.ready[0][sg], 0));
      r = transfers();
      if (r) return r;
      CU(cudaEventRecord(g.free_[0][sg], g.cs[0]));
    } else {
      if (k >= (u32)kvt_engine::N_STAGES) CU(cudaStreamWaitEvent(g.cs[1], g.free_[1][sg], 0));   // the stage was scattered
      r = transfers();
      if (r) return r;
      CU(cudaEventRecord(g.ready[1][sg], g.cs[1]));
      CU(cudaStreamWaitEvent(s, g.ready[1][sg], 0));
      r = launch_mover_views(e, s, stage_view(e, 1, sg, nb), nullptr, pool_view(e, dt), d_ids + b0, nb, nullptr, 0, false);
      if (r) return r;
      CU(cudaEventRecord(g.free_[1][sg], s));
    }
  }
  if (dir == 0)   // the caller's stream continues once the last transfers have landed
    for (u32 k = n_batches > (u32)kvt_engine::N_STAGES ? n_batches - kvt_engine::N_STAGES : 0; k < n_batches; ++k)
      CU(cudaStreamWaitEvent(s, g.free_[0][k % kvt_engine::N_STAGES], 0));
  if (timed) { CU(cudaEventRecord(e->ev_m1, s)); e->mover_timed = true; }
  return KVT_OK;
}

// Both directions at once through the staging ring: victims (HBM -> host) are gathered and sent on copy stream 0,
// reloads (host -> HBM) arrive and are scattered on copy stream 1, so both copy engines work. A reload may land in
// the HBM slot a victim of the same call leaves; payload copies are independent of the list order, so the victims
// are gathered in the order the reload batches need their slots, and the scatter of a batch waits for the gather
// of the last victim it depends on. All lists are host copies of what the plan kernels produced. When this
// returns, `s` waits for both copy streams.
int32_t staged_exchange(kvt_engine *e, cudaStream_t s, u32 n_in, const u32 *in_src, const u32 *in_dst, u32 n_out,
                        const u32 *out_src, const u32 *out_dst) {
  kvt_engine::Staging &g = e->stg;
  const u32 SB = g.blocks_per_stage;
  const u64 BB = e->block_bytes;
  const u32 NS = kvt_engine::N_STAGES;
  for (u32 i = 0; i < n_in; ++i) if (in_src[i] >= e->cfg.n_host_blocks) return fail(e, KVT_E_RANGE, "slot id out of range");
  for (u32 i = 0; i < n_out; ++i) if (out_dst[i] >= e->cfg.n_host_blocks) return fail(e, KVT_E_RANGE, "slot id out of range");
  const u32 nbi = cdiv(n_in, SB), nbo = cdiv(n_out, SB);
  // the reloads travel in the order of their host slots (long transfers); their HBM destinations follow that order
  std::vector<u32> in_order(n_in), in_src_s(n_in), in_dst_s(n_in);
  for (u32 i = 0; i < n_in; ++i) in_order[i] = i;
  std::sort(in_order.begin(), in_order.end(), [&](u32 x, u32 y) { return in_src[x] < in_src[y]; });
  for (u32 p = 0; p < n_in; ++p) { in_src_s[p] = in_src[in_order[p]]; in_dst_s[p] = in_dst[in_order[p]]; }
  in_src = in_src_s.data(); in_dst = in_dst_s.data();
  // order of the victims: those whose slots the first reload batches need come first
  std::map<u32, u32> vic_of;
  for (u32 v = 0; v < n_out; ++v) vic_of[out_src[v]] = v;
  std::vector<u32> order; order.reserve(n_out);
  std::vector<char> taken(n_out, 0);
  std::vector<u32> need(nbi, 0);
  for (u32 j = 0; j < nbi; ++j) {
    for (u32 r = j * SB; r < std::min(n_in, (j + 1) * SB); ++r) {
      auto it = vic_of.find(in_dst[r]);
      if (it != vic_of.end() && !taken[it->second]) { taken[it->second] = 1; order.push_back(it->second); }
    }
    need[j] = (u32)order.size();
  }
  for (u32 v = 0; v < n_out; ++v) if (!taken[v]) order.push_back(v);
  // device lists: victims' HBM slots in that order, and the place of every block inside its batch's stage (blocks
  // sit in the order of their host slots, so that consecutive host slots are one transfer)
  u32 *h_osrc = e->h_ids, *h_opos = e->h_ids2, *h_ipos = (u32 *)e->h_out, *h_idst = h_ipos + e->L.LB;
  u32 *d_osrc = e->dp<u32>(e->L.ids), *d_opos = e->dp<u32>(e->L.ids2), *d_ipos = e->dp<u32>(e->L.s0), *d_idst = e->dp<u32>(e->L.s1);
  std::vector<u32> ohost(n_out), isorted(n_in), osorted(n_out), idx(SB);
  for (u32 i = 0; i < n_out; ++i) { h_osrc[i] = out_src[order[i]]; ohost[i] = out_dst[order[i]]; }
  auto place = [&](const u32 *slots, u32 n, u32 *pos, std::vector<u32> &sorted) {
    for (u32 b0 = 0; b0 < n; b0 += SB) {
      const u32 nb = std::min(SB, n - b0);
      for (u32 i = 0; i < nb; ++i) idx[i] = i;
      std::sort(idx.begin(), idx.begin() + nb, [&](u32 x, u32 y) { return slots[b0 + x] < slots[b0 + y]; });
      for (u32 p = 0; p < nb; ++p) { pos[b0 + idx[p]] = p; sorted[b0 + p] = slots[b0 + idx[p]]; }
    }
  };
  place(ohost.data(), n_out, h_opos, osorted);
  place(in_src, n_in, h_ipos, isorted);
  for (u32 p = 0; p < n_in; ++p) h_idst[p] = in_dst[p];
  if (n_out) {
    CU(cudaMemcpyAsync(d_osrc, h_osrc, n_out * 4ull, cudaMemcpyHostToDevice, s));
    CU(cudaMemcpyAsync(d_opos, h_opos, n_out * 4ull, cudaMemcpyHostToDevice, s));
  }
  if (n_in) {
    CU(cudaMemcpyAsync(d_ipos, h_ipos, n_in * 4ull, cudaMemcpyHostToDevice, s));
    CU(cudaMemcpyAsync(d_idst, h_idst, n_in * 4ull, cudaMemcpyHostToDevice, s));
  }
  {
    int32_t r = stage_release(e, s);
    if (r) return r;
  }
  const bool timed = e->profiling;
  if (timed) CU(cudaEventRecord(e->ev_m0, s));
  CU(cudaEventRecord(g.begin, s));
  CU(cudaStreamWaitEvent(g.cs[0], g.begin, 0));
  CU(cudaStreamWaitEvent(g.cs[1], g.begin, 0));
  u8 *host_pool = (u8 *)e->cfg.host_pool;
  auto transfers = [&](int dir, const std::vector<u32> &sorted, u32 b0, u32 nb, u8 *stage) -> int32_t {
    for (u32 p = 0; p < nb;) {
      u32 run = 1;
      while (p + run < nb && sorted[b0 + p + run] == sorted[b0 + p] + run) ++run;
      u8 *hp = host_pool + (u64)sorted[b0 + p] * BB, *sp = stage + (u64)p * BB;
      if (dir == 0) CU(cudaMemcpyAsync(hp, sp, run * BB, cudaMemcpyDeviceToHost, g.cs[0]));
      else CU(cudaMemcpyAsync(sp, hp, run * BB, cudaMemcpyHostToDevice, g.cs[1]));
      p += run;
    }
    return KVT_OK;
  };
  auto issue_out = [&](u32 k) -> int32_t {   // gather + transfers of victim batch k, in order on copy stream 0
    const u32 b0 = k * SB, nb = std::min(SB, n_out - b0);
    const int sg = (int)(k % NS);
    int32_t r = launch_mover_views(e, g.cs[0], pool_view(e, KVT_TIER_HBM), d_osrc + b0, stage_view(e, 0, sg, nb), d_opos + b0, nb,
                                   nullptr, 0, false);
    if (r) return r;
    CU(cudaEventRecord(g.ready[0][sg], g.cs[0]));
    return transfers(0, osorted, b0, nb, stage_view(e, 0, sg, nb).base);
  };
  u32 ko = 0;
  for (u32 j = 0; j < nbi; ++j) {
    while (ko < nbo && ko * SB < need[j]) { int32_t r = issue_out(ko++); if (r) return r; }
    const u32 b0 = j * SB, nb = std::min(SB, n_in - b0);
    const int sg = (int)(j % NS);
    int32_t r = transfers(1, isorted, b0, nb, stage_view(e, 1, sg, nb).base);
    if (r) return r;
    if (need[j]) CU(cudaStreamWaitEvent(g.cs[1], g.ready[0][(ko - 1) % NS], 0));   // the victims in the way have been gathered
    r = launch_mover_views(e, g.cs[1], stage_view(e, 1, sg, nb), d_ipos + b0, pool_view(e, KVT_TIER_HBM), d_idst + b0, nb, nullptr, 0,
                           false);
    if (r) return r;
  }
  while (ko < nbo) { int32_t r = issue_out(ko++); if (r) return r; }
  CU(cudaEventRecord(g.free_[0][0], g.cs[0]));
  CU(cudaEventRecord(g.free_[1][0], g.cs[1]));
  CU(cudaStreamWaitEvent(s, g.free_[0][0], 0));
  CU(cudaStreamWaitEvent(s, g.free_[1][0], 0));
  if (timed) { CU(cudaEventRecord(e->ev_m1, s)); e->mover_timed = true; }
  return KVT_OK;
}

// After the stream has been synchronised: adds the timed mover kernel to the statistics.
void mover_account(kvt_engine *e, u64 blocks) {
  if (!e->mover_timed) return;
  e->mover_timed = false;
  float ms = 0.f;
  if (cudaEventElapsedTime(&ms, e->ev_m0, e->ev_m1) != cudaSuccess) return;
  e->st.mover_launches++;
  e->st.mover_ns += (u64)((double)ms * 1e6);
  e->st.mover_bytes += blocks * e->block_bytes;
}

// ---- classification -------------------------------------------------------------------------------------
constexpr int32_t INT_TBL_FULL = -100;   // internal: no room for the new message tables

// Message table of a context as it stands: the leading messages whose materialised bounds touch a mapped block.
u32 build_table(const Ctx &c, u32 *ms, u32 *me, u8 *mr, u32 cap) {
  u32 k = 0;
  for (size_t j = 0; j < c.mat_bounds.size(); ++j) {
    if (c.mat_bounds[j].first >= c.valid_blocks * 16ull) break;  // later messages touch no mapped block
    if (k >= cap) return 0xFFFFFFFFu;
    ms[k] = c.mat_bounds[j].first; me[k] = c.mat_bounds[j].second; mr[k] = msg_rank(c.msgs[j].state);
    ++k;
  }
  return k;
}

void snap_release(kvt_engine *e, Snap &sn) {
  if (sn.tbl_n) e->tbl_alloc.release(sn.tbl_off, sn.tbl_n);
  seg_deref(e, sn.keyseg);
  sn = Snap();
}

MsgTables msg_tables(kvt_engine *e) { return MsgTables{e->dp<u32>(e->L.m_start), e->dp<u32>(e->L.m_end), e->dp<u8>(e->L.m_rank)}; }

// Runs the delta kernel over the listed contexts (nullptr = a context that has ended: everything it was accounted
// for is taken away) and makes the current state what is accounted for. from_zero: the old side is empty for all.
int32_t apply_deltas(kvt_engine *e, cudaStream_t s, const std::vector<Ctx *> &list, std::vector<Snap> &ended, bool from_zero) {
  const u32 nd = (u32)(list.size() + ended.size());
  if (!nd) return KVT_OK;
  const u64 C = e->cfg.max_contexts, Mm = e->cfg.max_messages;
  if (nd > 2 * C) return fail(e, KVT_E_NOSPACE, "too many contexts ended since the last classification");
  DeltaCtx *hd = reinterpret_cast<DeltaCtx *>(e->h_desc + 2 * C * sizeof(SnapDesc));
  u32 nm = 0, nmap = 0, k = 0;
  std::vector<u32> tbl_n(list.size());
  for (size_t i = 0; i < list.size(); ++i) {
    const Ctx &c = *list[i];
    const bool maps = c.valid_blocks && c.keyseg >= 0;
    u32 n = maps ? build_table(c, e->h_mstart + nm, e->h_mend + nm, e->h_mrank + nm, (u32)Mm - nm) : 0;
    if (n == 0xFFFFFFFFu) return fail(e, KVT_E_NOSPACE, "max_messages exceeded");
    tbl_n[i] = n;
    nm += n;
  }
  u64 tbl_base = 0;
  if (nm && !e->tbl_alloc.alloc(nm, &tbl_base)) return INT_TBL_FULL;   // caller falls back to the full recomputation
  u32 off = 0;
  for (size_t i = 0; i < list.size(); ++i) {
    const Ctx &c = *list[i];
    const bool maps = c.valid_blocks && c.keyseg >= 0;
    const Snap &o = c.synced;
    DeltaCtx d{};
    if (!from_zero && o.keyseg >= 0) { d.old_key_off = e->segs[o.keyseg].off; d.old_valid = o.valid; d.old_tbl = (u32)o.tbl_off; d.old_n = o.tbl_n; }
    if (maps) { d.new_key_off = e->segs[c.keyseg].off; d.new_valid = c.valid_blocks; d.new_tbl = (u32)(tbl_base + off); d.new_n = tbl_n[i]; }
    d.map_base = nmap;
    nmap += std::max(d.old_valid, d.new_valid);
    off += tbl_n[i];
    hd[k++] = d;
  }
  for (const Snap &o : ended) {
    DeltaCtx d{};
    if (!from_zero && o.keyseg >= 0) { d.old_key_off = e->segs[o.keyseg].off; d.old_valid = o.valid; d.old_tbl = (u32)o.tbl_off; d.old_n = o.tbl_n; }
    d.map_base = nmap;
    nmap += d.old_valid;
    hd[k++] = d;
  }
  if (nmap) {
    DeltaCtx *dd = reinterpret_cast<DeltaCtx *>(e->dp<u8>(e->L.desc) + 2 * C * sizeof(SnapDesc));
    {
      SegCopy up(e, s);
      up.add(dd, hd, nd * sizeof(DeltaCtx));
      up.add(e->dp<u32>(e->L.m_start) + tbl_base, e->h_mstart, nm * 4ull);
      up.add(e->dp<u32>(e->L.m_end) + tbl_base, e->h_mend, nm * 4ull);
      up.add(e->dp<u8>(e->L.m_rank) + tbl_base, e->h_mrank, nm);
      up.flush();
    }
    DeltaArgs a;
    a.tab = e->tab; a.ent = e->ent; a.keys = e->d_keys; a.ctx = dd; a.n_ctx = nd; a.n_map = nmap; a.tbl = msg_tables(e);
    a.status = e->d_status; a.first_miss = nullptr;
    if (from_zero && (e->cfg.policy_flags & KVT_POLICY_ORPHANS_DEAD)) {
      a.first_miss = e->dp<u32>(e->L.freelist2);   // scratch of the list calls, free between calls (stream order)
      if (nd > e->L.LB) return fail(e, KVT_E_NOSPACE, "more contexts than max_batch_blocks");
      CU(cudaMemsetAsync(a.first_miss, 0xFF, nd * 4ull, s));
      KLM(k_first_miss, cdiv(nmap, TPB), TPB, s, a);
    }
    const bool timed = e->profiling && !e->classify_timed;
    if (timed) CU(cudaEventRecord(e->ev_c0, s));
    KLM(k_map_delta, cdiv(nmap, TPB), TPB, s, a);
    if (timed) { CU(cudaEventRecord(e->ev_c1, s)); e->classify_timed = true; e->classify_pending_items = nmap; }
    LAUNCH_CHECK();
  }
  // what is accounted for now
  off = 0;
  for (size_t i = 0; i < list.size(); ++i) {
    Ctx &c = *list[i];
    const bool maps = c.valid_blocks && c.keyseg >= 0;
    Snap n;
    if (maps) { n.keyseg = c.keyseg; e->segs[c.keyseg].refs++; n.valid = c.valid_blocks; n.tbl_off = tbl_base + off; n.tbl_n = tbl_n[i]; }
    off += tbl_n[i];
    snap_release(e, c.synced);
    c.synced = n;
    c.map_dirty = false;
  }
  for (Snap &o : ended) snap_release(e, o);
  ended.clear();
  return KVT_OK;
}

// Recomputes every count from zero over all contexts.
int32_t full_recount(kvt_engine *e, cudaStream_t s) {
  for (Ctx &c : e->ctxs) if (c.live) snap_release(e, c.synced);
  for (Snap &o : e->zombies) snap_release(e, o);
  e->zombies.clear();
  e->tbl_alloc.init(2ull * e->cfg.max_messages, 1);
  CU(cudaMemsetAsync(e->ent.cnt, 0, (u64)e->ent.n_total * 8, s));
  std::vector<Ctx *> all;
  for (Ctx &c : e->ctxs) if (c.live) all.push_back(&c);
  int32_t r = apply_deltas(e, s, all, e->zombies, true);
  return r == INT_TBL_FULL ? fail(e, KVT_E_NOSPACE, "max_messages exceeded") : r;
}

// Brings the per-block mapping counts up to date with everything that happened since the last time.
int32_t do_classify(kvt_engine *e, cudaStream_t s, bool force_full = false) {
  int32_t r = stage_acquire(e);
  if (r) return r;
  const bool full = force_full || e->full_dirty || e->classify_mode == 1 || (e->cfg.policy_flags & KVT_POLICY_ORPHANS_DEAD);
  if (full) {
    r = full_recount(e, s);
    if (r) return r;
  } else {
    const u64 C = e->cfg.max_contexts;
    // (1) entries inserted since then get the contributions of every mapping already accounted for
    if (e->n_fresh) {
      SnapDesc *hs = reinterpret_cast<SnapDesc *>(e->h_desc);
      u32 ns = 0;
      auto add = [&](const Snap &o) {
        if (o.keyseg < 0 || !o.valid || ns >= 2 * C) return;
        hs[ns++] = SnapDesc{e->segs[o.keyseg].off, o.valid, (u32)o.tbl_off, o.tbl_n, 0};
      };
      for (const Ctx &c : e->ctxs) if (c.live) add(c.synced);
      for (const Snap &o : e->zombies) add(o);
      if (ns) {
        SnapDesc *ds = reinterpret_cast<SnapDesc *>(e->dp<u8>(e->L.desc));
        { SegCopy up(e, s); up.add(ds, hs, ns * sizeof(SnapDesc)); up.flush(); }
        FixArgs a;
        a.tab = e->tab; a.ent = e->ent; a.keys = e->d_keys; a.snaps = ds; a.n_snaps = ns; a.tbl = msg_tables(e);
        a.fresh = e->dp<u32>(e->L.fresh); a.n_fresh = e->n_fresh; a.status = e->d_status;
        KLM(k_fresh_fixup, cdiv(e->n_fresh, 128), 128, s, a);
      }
    }
    // (2) contexts that changed, and contexts that ended
    std::vector<Ctx *> list;
    for (Ctx &c : e->ctxs) if (c.live && c.map_dirty) list.push_back(&c);
    r = apply_deltas(e, s, list, e->zombies, false);
    if (r == INT_TBL_FULL) r = full_recount(e, s);   // the table arena is fragmented or full: start over
    if (r) return r;
  }
  e->n_fresh = 0;
  r = stage_release(e, s);
  if (r) return r;
  LAUNCH_CHECK();
  e->dirty = false;
  e->full_dirty = false;
  if (e->classify_mode == 2 && !full) {   // cross-check: the event-driven counts must equal a full recomputation
    CU(cudaMemcpyAsync(e->dp<u64>(e->L.cnt_chk), e->ent.cnt, (u64)e->ent.n_total * 8, cudaMemcpyDeviceToDevice, s));
    r = do_classify(e, s, true);
    if (r) return r;
    CU(cudaMemsetAsync(e->d_status + ST_CHK, 0, 4, s));
    KL(k_cnt_compare, cdiv(e->ent.n_total, TPB), TPB, s, e->dp<u64>(e->L.cnt_chk), e->ent.cnt, e->ent.n_total, e->d_status + ST_CHK);
    LAUNCH_CHECK();
    CU(cudaMemcpyAsync(e->h_status + ST_CHK, e->d_status + ST_CHK, 4, cudaMemcpyDeviceToHost, s));
    CU(cudaStreamSynchronize(s));
    if (e->h_status[ST_CHK]) return fail(e, KVT_E_DEVICE, "event-driven classification differs from the full recomputation");
  }
  return KVT_OK;
}

int32_t ensure_classified(kvt_engine *e, cudaStream_t s) { return e->dirty ? do_classify(e, s) : KVT_OK; }

// A context ends: what is accounted for it is kept until the next classification takes it away.
int32_t retire_ctx(kvt_engine *e, Ctx &c, cudaStream_t s) {
  if (c.synced.keyseg >= 0 && c.synced.valid) {
    if (e->zombies.size() >= e->cfg.max_contexts) {   // bounded: bring the counts up to date first
      c.map_dirty = true;
      int32_t r = do_classify(e, s);
      if (r) return r;
    }
    e->zombies.push_back(c.synced);
    c.synced = Snap();
  } else {
    snap_release(e, c.synced);
  }
  seg_deref(e, c.keyseg);
  c = Ctx();
  return KVT_OK;
}

// ---- token buffers ---------------------------------------------------------------------------------------
int32_t copy_tokens_in(kvt_engine *e, cudaStream_t s, u64 dst_tok, const u32 *src, u32 n, bool on_device) {
  if (!n) return KVT_OK;
  CU(cudaMemcpyAsync(e->d_tokens + dst_tok, src, (u64)n * 4, on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, s));
  return KVT_OK;
}

int32_t copy_tokens_dd(kvt_engine *e, cudaStream_t s, u64 dst_tok, u64 src_tok, u64 n) {
  if (!n) return KVT_OK;
  CU(cudaMemcpyAsync(e->d_tokens + dst_tok, e->d_tokens + src_tok, n * 4, cudaMemcpyDeviceToDevice, s));
  return KVT_OK;
}

u64 grow_cap(u64 need) { return round_up(std::max<u64>(need + need / 4, 1024), 64); }

int32_t unlock_held(kvt_engine *e, Ctx &c, cudaStream_t s, bool stamp) {
  if (c.held && c.keyseg >= 0) {
    KLM(k_unlock, cdiv(c.held, TPB), TPB, s, e->tab, e->ent, (const u64 *)(e->d_keys + e->segs[c.keyseg].off), c.held, e->now,
        stamp ? 1u : 0u, e->d_status);
    LAUNCH_CHECK();
  }
  c.held = 0;
  return KVT_OK;
}

// Index of the first block >= from made only of Temporary tokens, or n_blocks (Algorithm 1's bypass).
u32 first_temporary_block(const Ctx &c, u32 from, u32 n_blocks) {
  u64 pos = 0;
  bool in_run = false;
  u64 run_s = 0;
  auto close_run = [&](u64 run_e) -> u32 {
    u64 b0 = std::max<u64>((run_s + 15) / 16, from), b1 = run_e / 16;  // blocks fully inside [run_s, run_e)
    if (b0 < b1 && b0 < n_blocks) return (u32)b0;
    return 0xFFFFFFFFu;
  };
  for (const Msg &m : c.msgs) {
    if (m.len) {
      bool temp = msg_rank(m.state) == 0;
      if (temp && !in_run) { in_run = true; run_s = pos; }
      if (!temp && in_run) { in_run = false; u32 b = close_run(pos); if (b != 0xFFFFFFFFu) return b; }
    }
    pos += m.len;
  }
  if (in_run) { u32 b = close_run(pos); if (b != 0xFFFFFFFFu) return b; }
  return n_blocks;
}

// Blocks in [from, to) touched by a non-empty Pinned message.
u32 count_pinned_blocks(const Ctx &c, u32 from, u32 to) {
  u64 pos = 0;
  u32 n = 0;
  int64_t last = -1;   // last block already counted
  for (const Msg &m : c.msgs) {
    if (m.len && m.state == MS_PINNED) {
      int64_t b0 = std::max<int64_t>((int64_t)(pos / 16), std::max<int64_t>(from, last + 1));
      int64_t b1 = std::min<int64_t>((int64_t)((pos + m.len - 1) / 16), (int64_t)to - 1);
      if (b1 >= b0) { n += (u32)(b1 - b0 + 1); last = b1; }
    }
    pos += m.len;
  }
  return n;
}

}  // namespace

// =========================================================================================================
// C ABI
// =========================================================================================================
extern "C" {

int32_t kvt_query_sizes(const kvt_config *cfg, uint64_t *meta_bytes, uint64_t *token_bytes) {
  if (!cfg || !meta_bytes || !token_bytes) return KVT_E_INVAL;
  *meta_bytes = make_layout(*cfg).total;
  *token_bytes = round_up(cfg->max_tokens * 4, 256);
  return KVT_OK;
}

int32_t kvt_create(const kvt_config *cfg, void *stream, kvt_engine **out) {
  if (!cfg || !out) return KVT_E_INVAL;
  const kvt_config &c = *cfg;
  if (c.abi_version != KVT_ABI_VERSION || c.block_tokens != 16 || !c.n_layers || !c.n_kv_heads || !c.head_dim ||
      !c.elem_bytes || c.pool_layout > 1 || !c.n_hbm_blocks || !c.max_contexts || !c.max_batch_blocks ||
      !c.max_messages || c.suspended_order > 1 || c.policy_flags > 7 || !c.dev_meta || !c.dev_tokens)
    return KVT_E_INVAL;
  u64 N = (u64)c.n_hbm_blocks + c.n_host_blocks + c.n_remote_blocks;
  if (N >= CLAIM_BIT || c.max_batch_blocks >= CLAIM_BIT) return KVT_E_INVAL;
  if (c.table_capacity < 2 * N || (c.table_capacity & (c.table_capacity - 1))) return KVT_E_INVAL;
  if (((uintptr_t)c.dev_meta & 255) || ((uintptr_t)c.dev_tokens & 255)) return KVT_E_INVAL;
  DevLayout L = make_layout(c);
  if (c.dev_meta_bytes < L.total || c.dev_tokens_bytes < c.max_tokens * 4) return KVT_E_INVAL;
  u64 chunk_bytes = 16ull * c.n_kv_heads * c.head_dim * c.elem_bytes, n_chunks = 2ull * c.n_layers;
  bool meta_only = c.hbm_pool == nullptr;
  if (!meta_only) {
    if (c.stage_buf && ((uintptr_t)c.stage_buf & 15)) return KVT_E_INVAL;
    if (c.hbm_pool_bytes < chunk_bytes * n_chunks * c.n_hbm_blocks || ((uintptr_t)c.hbm_pool & 15)) return KVT_E_INVAL;
    if (c.n_host_blocks && (!c.host_pool || c.host_pool_bytes < chunk_bytes * n_chunks * c.n_host_blocks ||
                            ((uintptr_t)c.host_pool & 15)))
      return KVT_E_INVAL;
    if (c.n_remote_blocks && (!c.remote_pool || c.remote_pool_bytes < chunk_bytes * n_chunks * c.n_remote_blocks ||
                              ((uintptr_t)c.remote_pool & 15)))
      return KVT_E_INVAL;
  }
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return KVT_E_CUDA;
  kvt_engine *e = new kvt_engine();
  e->cfg = c; e->L = L;
  e->meta = (u8 *)c.dev_meta; e->d_tokens = (u32 *)c.dev_tokens;
  e->chunk_bytes = chunk_bytes; e->n_chunks = n_chunks; e->block_bytes = chunk_bytes * n_chunks;
  e->metadata_only = meta_only;
  if (!meta_only) {
    const void *pools[3] = {c.hbm_pool, c.n_host_blocks ? c.host_pool : nullptr, c.n_remote_blocks ? c.remote_pool : nullptr};
    for (int t = 0; t < 3; ++t) {
      cudaPointerAttributes at;
      if (pools[t] && cudaPointerGetAttributes(&at, pools[t]) == cudaSuccess) e->tier_in_host_mem[t] = at.type == cudaMemoryTypeHost;
      else cudaGetLastError();
    }
  }
  cudaDeviceGetAttribute(&e->sm_count, cudaDevAttrMultiProcessorCount, dev);
  if (!meta_only && c.stage_buf && c.stage_bytes) {
    kvt_engine::Staging &g = e->stg;
    g.buf = (u8 *)c.stage_buf;
    g.blocks_per_stage = (u32)std::min<u64>(c.stage_bytes / (2ull * kvt_engine::N_STAGES) / e->block_bytes, 0x7FFFFFFFu);
    bool okk = g.blocks_per_stage > 0;
    for (int d = 0; d < 2 && okk; ++d) {
      okk = cudaStreamCreateWithFlags(&g.cs[d], cudaStreamNonBlocking) == cudaSuccess;
      for (int k = 0; k < kvt_engine::N_STAGES && okk; ++k)
        okk = cudaEventCreateWithFlags(&g.ready[d][k], cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&g.free_[d][k], cudaEventDisableTiming) == cudaSuccess;
    }
    okk = okk && cudaEventCreateWithFlags(&g.begin, cudaEventDisableTiming) == cudaSuccess;
    if (!okk) cudaGetLastError();
    g.ok = okk;
  }
  e->tab.slots = e->dp<TSlot>(L.tab); e->tab.mask = c.table_capacity - 1;
  e->tab.shift = 64 - (bit_length(c.table_capacity) - 1);
  e->ent.key = e->dp<u64>(L.e_key); e->ent.stamp = e->dp<u32>(L.e_stamp); e->ent.depth = e->dp<u32>(L.e_depth);
  e->ent.infl = e->dp<u32>(L.e_infl); e->ent.cnt = e->dp<u64>(L.e_cnt); e->ent.tslot = e->dp<u32>(L.e_tslot);
  e->ent.mark = e->dp<u32>(L.e_mark); e->ent.floor = e->dp<u8>(L.e_floor); e->ent.link = e->dp<u32>(L.e_link);
  e->ent.n_hbm = c.n_hbm_blocks; e->ent.n_host = c.n_host_blocks; e->ent.n_total = (u32)N;
  e->d_keys = e->dp<u64>(L.keys); e->d_status = e->dp<u32>(L.status);
  e->h0 = hash_h0(c.hash_seed);
  {   // L2 residency window: table, keys, stamps, depths, in-flight counts, mapping counts (contiguous in the arena)
    int max_persist = 0, max_win = 0;
    cudaDeviceGetAttribute(&max_persist, cudaDevAttrMaxPersistingL2CacheSize, dev);
    cudaDeviceGetAttribute(&max_win, cudaDevAttrMaxAccessPolicyWindowSize, dev);
    const u64 bytes = std::min<u64>(L.e_tslot - L.tab, (u64)std::max(max_win, 0));
    const u64 want = std::min<u64>(bytes, (u64)std::max(max_persist, 0));
    size_t cur = 0;
    if (bytes && want && cudaDeviceGetLimit(&cur, cudaLimitPersistingL2CacheSize) == cudaSuccess &&
        (cur >= want || cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, want) == cudaSuccess)) {
      e->l2_win.base_ptr = e->meta + L.tab;
      e->l2_win.num_bytes = bytes;
      e->l2_win.hitRatio = (float)std::min(1.0, (double)want / (double)bytes);
      e->l2_win.hitProp = cudaAccessPropertyPersisting;
      e->l2_win.missProp = cudaAccessPropertyNormal;
      e->l2_on = true;
    } else {
      cudaGetLastError();
    }
  }
  e->ctxs.resize(c.max_contexts);
  e->tok_alloc.init(c.max_tokens, 64);
  e->key_alloc.init(c.max_key_blocks + c.max_key_blocks / CHUNK + 64ull * c.max_contexts, 32);
  e->tbl_alloc.init(2ull * c.max_messages, 1);
  // pinned staging
  u64 C = c.max_contexts, Mm = c.max_messages, LB = L.LB;
  u64 o_status = 0, o_ctxres = L.ctxres - L.status, o_desc = L.desc - L.status,
      o_ms = o_desc + round_up(C * 256 + 2 * (c.max_batch_blocks / CHUNK + C + 1) * 4, 256),
      o_me = o_ms + round_up(Mm * 4, 256), o_mr = o_me + round_up(Mm * 4, 256), o_ids = o_mr + round_up(Mm, 256),
      o_ids2 = o_ids + round_up(LB * 4, 256), o_out = o_ids2 + round_up(LB * 4, 256),
      o_sel = o_out + round_up(LB * 16, 256), total = o_sel + round_up(sizeof(SelArgs), 256);
  if (cudaHostAlloc((void **)&e->stage, total, cudaHostAllocDefault) != cudaSuccess) { delete e; return KVT_E_CUDA; }
  e->h_status = (u32 *)(e->stage + o_status); e->h_desc = e->stage + o_desc; e->h_ctxres = (u32 *)(e->stage + o_ctxres);
  e->h_mstart = (u32 *)(e->stage + o_ms); e->h_mend = (u32 *)(e->stage + o_me); e->h_mrank = e->stage + o_mr;
  e->h_ids = (u32 *)(e->stage + o_ids); e->h_ids2 = (u32 *)(e->stage + o_ids2); e->h_out = e->stage + o_out;
  e->h_sel = (SelArgs *)(e->stage + o_sel);
  cudaStream_t s = (cudaStream_t)stream;
  if (cudaStreamCreateWithFlags(&e->capture_stream, cudaStreamNonBlocking) != cudaSuccess) { cudaGetLastError(); e->use_graphs = false; }
#ifdef KVT_TRACE
  if (getenv("KVT_NO_OVERLAP")) e->overlap_launches = false;
  if (getenv("KVT_NO_GRAPH")) e->use_graphs = false;
#endif
  if (CHECKED_BUILD) e->use_graphs = false;
  bool ok = cudaEventCreateWithFlags(&e->ev_upload, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreate(&e->ev_m0) == cudaSuccess && cudaEventCreate(&e->ev_m1) == cudaSuccess &&
            cudaEventCreate(&e->ev_h0) == cudaSuccess && cudaEventCreate(&e->ev_h1) == cudaSuccess &&
            cudaEventCreate(&e->ev_c0) == cudaSuccess && cudaEventCreate(&e->ev_c1) == cudaSuccess;
  // everything except the key arena and scratch must start at zero; the table needs ent = NONE
  ok = ok && cudaMemsetAsync(e->meta + L.e_key, 0, L.keys - L.e_key, s) == cudaSuccess;
  ok = ok && cudaMemsetAsync(e->d_status, 0, ST_WORDS * 4, s) == cudaSuccess;
  ok = ok && cudaMemsetAsync(e->ent.link, 0xFF, N * 4, s) == cudaSuccess;   // no links
  if (ok) {
    KL(k_table_clear, cdiv((u64)c.table_capacity, TPB), TPB, s, e->tab);
    ok = cudaGetLastError() == cudaSuccess && cudaStreamSynchronize(s) == cudaSuccess;
  }
  if (!ok) { cudaFreeHost(e->stage); if (e->ev_upload) cudaEventDestroy(e->ev_upload); delete e; return KVT_E_CUDA; }
  *out = e;
  return KVT_OK;
}

int32_t kvt_destroy(kvt_engine *e) {
  if (!e) return KVT_E_INVAL;
  cudaDeviceSynchronize();
  if (e->l2_win.num_bytes) cudaCtxResetPersistingL2Cache();   // the lines this engine kept resident are ordinary lines again
  for (auto &m : e->sel_graph) for (auto &g : m) if (g.second.exec) cudaGraphExecDestroy(g.second.exec);
  if (e->capture_stream) cudaStreamDestroy(e->capture_stream);
  for (int d = 0; d < 2; ++d) {
    if (e->stg.cs[d]) cudaStreamDestroy(e->stg.cs[d]);
    for (int k = 0; k < kvt_engine::N_STAGES; ++k) {
      if (e->stg.ready[d][k]) cudaEventDestroy(e->stg.ready[d][k]);
      if (e->stg.free_[d][k]) cudaEventDestroy(e->stg.free_[d][k]);
    }
  }
  if (e->stg.begin) cudaEventDestroy(e->stg.begin);
  if (e->ev_upload) cudaEventDestroy(e->ev_upload);
  if (e->ev_m0) cudaEventDestroy(e->ev_m0);
  if (e->ev_m1) cudaEventDestroy(e->ev_m1);
  if (e->ev_h0) cudaEventDestroy(e->ev_h0);
  if (e->ev_h1) cudaEventDestroy(e->ev_h1);
  if (e->ev_c0) cudaEventDestroy(e->ev_c0);
  if (e->ev_c1) cudaEventDestroy(e->ev_c1);
  if (e->stage) cudaFreeHost(e->stage);
  delete e;
  return KVT_OK;
}

int32_t kvt_last_error(kvt_engine *e, char *buf, uint32_t cap) {
  if (!e || !buf || !cap) return KVT_E_INVAL;
  std::snprintf(buf, cap, "%s", e->err.c_str());
  return KVT_OK;
}

int32_t kvt_set_profiling(kvt_engine *e, uint32_t on) {
  if (!e) return KVT_E_INVAL;
  e->profiling = on != 0;
  return KVT_OK;
}

int32_t kvt_debug_set_mover_variant(kvt_engine *e, uint32_t variant) {
  if (!e) return KVT_E_INVAL;
  if (variant > 4) return KVT_E_INVAL;
  e->mover_variant = variant;
  return KVT_OK;
}

int32_t kvt_set_mover_ctas(kvt_engine *e, uint32_t max_ctas) {
  if (!e) return KVT_E_INVAL;
  e->mover_max_ctas = max_ctas;
  return KVT_OK;
}

int32_t kvt_debug_set_lookup_variant(kvt_engine *e, uint32_t variant) {
  if (!e || variant > 4) return KVT_E_INVAL;
  e->lookup_variant = variant;
  return KVT_OK;
}

int32_t kvt_set_l2_residency(kvt_engine *e, uint32_t on) {
  if (!e) return KVT_E_INVAL;
  if (on && !e->l2_win.num_bytes) return fail(e, KVT_E_INVAL, "this device offers no persisting L2");
  e->l2_on = on != 0;
  if (!on) cudaCtxResetPersistingL2Cache();
  return KVT_OK;
}

int32_t kvt_debug_set_copy_delay(kvt_engine *e, uint32_t delay_ns) {
  if (!e || delay_ns > 1000000u) return KVT_E_INVAL;
  e->copy_delay_ns = delay_ns;
  return KVT_OK;
}

int32_t kvt_debug_set_classify_mode(kvt_engine *e, uint32_t mode) {
  if (!e || mode > 2) return KVT_E_INVAL;
  e->classify_mode = mode;
  return KVT_OK;
}

int32_t kvt_debug_set_wait_limit(kvt_engine *e, uint32_t polls) {
  if (!e) return KVT_E_INVAL;
  e->wait_limit = polls;
  return KVT_OK;
}

int32_t kvt_get_stats(kvt_engine *e, kvt_stats *out) {
  if (!e || !out) return KVT_E_INVAL;
  if (e->classify_timed && cudaEventQuery(e->ev_c1) == cudaSuccess) {   // classification is asynchronous: its time is read here
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, e->ev_c0, e->ev_c1) == cudaSuccess) {
      e->st.classify_ns += (u64)((double)ms * 1e6); e->st.classify_items += e->classify_pending_items;
    }
    e->classify_timed = false;
  }
  kvt_stats s = e->st;
  s.clock = e->now;
  s.n_contexts = 0;
  for (const Ctx &c : e->ctxs) s.n_contexts += c.live;
  s.occ_hbm = e->occ[0]; s.occ_host = e->occ[1]; s.occ_remote = e->occ[2];
  s.tombstones = e->tombs;
  *out = s;
  return KVT_OK;
}

// ---- stage 0 -----------------------------------------------------------------------------------------------
int32_t kvt_apply_op(kvt_engine *e, const kvt_op *op, void *stream) {
  if (!e || !op) return KVT_E_INVAL;
  cudaStream_t s = (cudaStream_t)stream;
  const u32 id = op->ctx;
  const bool on_dev = op->flags & KVT_OPF_TOKENS_ON_DEVICE;
  if (op->op == KVT_OP_SPAWN) {
    if (id >= e->ctxs.size() || e->ctxs[id].live) return fail(e, KVT_E_INVAL, "spawn: context id out of range or in use");
    e->ctxs[id] = Ctx();
    e->ctxs[id].live = true;
    return KVT_OK;
  }
  if (op->op == KVT_OP_FORK) {
    if (id >= e->ctxs.size() || e->ctxs[id].live) return fail(e, KVT_E_INVAL, "fork: child id out of range or in use");
    Ctx *p = get_ctx(e, op->parent);
    if (!p) return fail(e, KVT_E_NOCTX, "fork: unknown parent");
    if (p->in_flight) return fail(e, KVT_E_STATE, "fork: parent is in flight");
    if (op->msg_end > p->msgs.size()) return fail(e, KVT_E_RANGE, "fork: end beyond the parent's messages");
    Ctx k;
    k.live = true;
    u64 T = 0;
    for (u32 j = 0; j < op->msg_end; ++j) { k.msgs.push_back(Msg{p->msgs[j].len, (u8)MS_ACTIVE}); T += p->msgs[j].len; }
    k.tok_cap = grow_cap(T);
    if (!e->tok_alloc.alloc(k.tok_cap, &k.tok_off)) return fail(e, KVT_E_NOSPACE, "token arena full");
    k.tok_len = T;
    if (T) {
      cudaError_t ce = cudaMemcpyAsync(e->d_tokens + k.tok_off, e->d_tokens + p->tok_off, T * 4, cudaMemcpyDeviceToDevice, s);
      if (ce != cudaSuccess) { e->tok_alloc.release(k.tok_off, k.tok_cap); e->err = cudaGetErrorString(ce); return KVT_E_CUDA; }
    }
    u32 m = std::min<u32>(op->msg_end, (u32)p->mat_bounds.size());
    u32 Tm = m ? p->mat_bounds[m - 1].second : 0;
    k.mat_bounds.assign(p->mat_bounds.begin(), p->mat_bounds.begin() + m);
    k.mat_blocks = Tm / 16;
    k.valid_blocks = std::min<u32>(Tm / 16, p->valid_blocks);
    if (k.mat_blocks && p->keyseg >= 0) { k.keyseg = p->keyseg; e->segs[p->keyseg].refs++; }  // equal prefixes, equal keys
    else { k.mat_blocks = 0; k.valid_blocks = 0; }
    k.map_dirty = true;
    e->ctxs[id] = std::move(k);
    e->dirty = true;
    return KVT_OK;
  }
  if (op->op == 0 || op->op > KVT_OP_UNPIN) return fail(e, KVT_E_INVAL, "unknown op");
  Ctx *c = get_ctx(e, id, op->op == KVT_OP_UNPIN);   // a terminated context kept for its Pinned messages only accepts unpin
  if (!c) return fail(e, KVT_E_NOCTX, "unknown context");
  switch (op->op) {
    case KVT_OP_APPEND: {
      if (c->in_flight) return fail(e, KVT_E_STATE, "append: context is in flight");
      if (op->n_tokens && !op->tokens) return fail(e, KVT_E_INVAL, "append: NULL tokens");
      u64 need = c->tok_len + op->n_tokens;
      if (need > c->tok_cap) {
        u64 ncap = grow_cap(std::max<u64>(need, 2 * c->tok_cap)), noff;
        if (!e->tok_alloc.alloc(ncap, &noff)) return fail(e, KVT_E_NOSPACE, "token arena full");
        int32_t r = copy_tokens_dd(e, s, noff, c->tok_off, c->tok_len);
        if (!r) r = copy_tokens_in(e, s, noff + c->tok_len, op->tokens, op->n_tokens, on_dev);
        if (r) { e->tok_alloc.release(noff, ncap); return r; }   // the context keeps its old buffer
        if (c->tok_cap) e->tok_alloc.release(c->tok_off, c->tok_cap);
        c->tok_off = noff; c->tok_cap = ncap;
      } else {
        int32_t r = copy_tokens_in(e, s, c->tok_off + c->tok_len, op->tokens, op->n_tokens, on_dev);
        if (r) return r;
      }
      c->tok_len = need;
      c->msgs.push_back(Msg{op->n_tokens, (u8)(c->one_off ? MS_TEMPORARY : MS_ACTIVE)});   // no KV effect before the next call
      return KVT_OK;
    }
    case KVT_OP_REPLACE:
    case KVT_OP_REMOVE: {
      if (c->in_flight) return fail(e, KVT_E_STATE, "edit: context is in flight");
      if (!(op->msg_start < op->msg_end && op->msg_end <= c->msgs.size())) return fail(e, KVT_E_RANGE, "edit: bad message range");
      const bool rep = op->op == KVT_OP_REPLACE;
      if (rep && op->n_tokens && !op->tokens) return fail(e, KVT_E_INVAL, "replace: NULL tokens");
      u64 t0 = 0, t1 = 0;
      for (u32 j = 0; j < op->msg_end; ++j) { if (j < op->msg_start) t0 += c->msgs[j].len; t1 += c->msgs[j].len; }
      const u64 nnew = rep ? op->n_tokens : 0, tail = c->tok_len - t1, new_len = t0 + nnew + tail;
      if (tail == 0 && t0 + nnew <= c->tok_cap) {  // edit at the end: overwrite in place
        int32_t r = copy_tokens_in(e, s, c->tok_off + t0, op->tokens, (u32)nnew, on_dev);
        if (r) return r;
      } else {                                      // edit in the middle: rebuild the buffer elsewhere
        u64 ncap = grow_cap(new_len), noff;
        if (!e->tok_alloc.alloc(ncap, &noff)) return fail(e, KVT_E_NOSPACE, "token arena full");
        int32_t r = copy_tokens_dd(e, s, noff, c->tok_off, t0);
        if (!r) r = copy_tokens_in(e, s, noff + t0, op->tokens, (u32)nnew, on_dev);
        if (!r) r = copy_tokens_dd(e, s, noff + t0 + nnew, c->tok_off + t1, tail);
        if (r) { e->tok_alloc.release(noff, ncap); return r; }   // the context keeps its old buffer
        if (c->tok_cap) e->tok_alloc.release(c->tok_off, c->tok_cap);
        c->tok_off = noff; c->tok_cap = ncap;
      }
      c->tok_len = new_len;
      // the old versions of message msg_start and of all later messages expire for this context:
      // it stops mapping everything from the block holding that message's first token (Section 5.1)
      if (op->msg_start < c->mat_bounds.size()) {
        c->valid_blocks = std::min<u32>(c->valid_blocks, c->mat_bounds[op->msg_start].first / 16);
        c->mat_bounds.resize(op->msg_start);
      }
      c->msgs.erase(c->msgs.begin() + op->msg_start, c->msgs.begin() + op->msg_end);
      if (rep) c->msgs.insert(c->msgs.begin() + op->msg_start, Msg{op->n_tokens, (u8)(c->one_off ? MS_TEMPORARY : MS_ACTIVE)});
      c->map_dirty = true;
      e->dirty = true;
      return KVT_OK;
    }
    case KVT_OP_ONE_OFF: {
      if (c->in_flight) return fail(e, KVT_E_STATE, "one_off: context is in flight");
      if (op->msg_start == 0 && op->msg_end == 0xFFFFFFFFu) {
        c->one_off = true;
        for (Msg &m : c->msgs) if (m.state != MS_PINNED) m.state = MS_TEMPORARY;   // explicit protection stays
      } else {
        if (!(op->msg_start < op->msg_end && op->msg_end <= c->msgs.size())) return fail(e, KVT_E_RANGE, "one_off: bad message range");
        for (u32 j = op->msg_start; j < op->msg_end; ++j) c->msgs[j].state = MS_TEMPORARY;
      }
      c->map_dirty = true;
      e->dirty = true;
      return KVT_OK;
    }
    case KVT_OP_PREFILL_DONE: {
      if (!c->in_flight) return fail(e, KVT_E_STATE, "prefill_done: context is not in flight");
      if (e->now == 0xFFFFFFFFu) return fail(e, KVT_E_NOSPACE, "logical clock exhausted");
      e->now += 1;
      int32_t r = unlock_held(e, *c, s, true);
      if (r) return r;
      for (Msg &m : c->msgs) if (m.state == MS_ACTIVE) m.state = MS_SUSPENDED;
      c->in_flight = false;
      c->map_dirty = true;
      e->dirty = true;
      return KVT_OK;
    }
    case KVT_OP_TERMINATE: {
      if (c->in_flight) { int32_t r = unlock_held(e, *c, s, false); if (r) return r; }
      if (c->tok_cap) e->tok_alloc.release(c->tok_off, c->tok_cap);
      c->tok_off = c->tok_cap = c->tok_len = 0;
      bool pinned = false;
      for (Msg &m : c->msgs) { if (m.state == MS_PINNED) pinned = true; else m.state = MS_EXPIRED; }
      e->dirty = true;
      if (pinned) {            // Pinned messages retain their protection: keep the mapping, drop the rest
        c->terminated = true;
        c->in_flight = false;
        c->map_dirty = true;
      } else {
        return retire_ctx(e, *c, s);
      }
      return KVT_OK;
    }
    case KVT_OP_PIN:
    case KVT_OP_UNPIN: {
      if (c->in_flight) return fail(e, KVT_E_STATE, "pin/unpin: context is in flight");
      if (!(op->msg_start < op->msg_end && op->msg_end <= c->msgs.size())) return fail(e, KVT_E_RANGE, "pin/unpin: bad message range");
      for (u32 j = op->msg_start; j < op->msg_end; ++j) {
        Msg &m = c->msgs[j];
        if (op->op == KVT_OP_PIN) m.state = MS_PINNED;
        else if (m.state == MS_PINNED) m.state = c->terminated ? MS_EXPIRED : (c->one_off ? MS_TEMPORARY : MS_SUSPENDED);
      }
      if (c->terminated) {
        bool pinned = false;
        for (const Msg &m : c->msgs) pinned = pinned || m.state == MS_PINNED;
        if (!pinned) { e->dirty = true; return retire_ctx(e, *c, s); }
      }
      c->map_dirty = true;
      e->dirty = true;
      return KVT_OK;
    }
  }
  return KVT_E_INVAL;
}

// ---- stages 1 + 2 + admission ---------------------------------------------------------------------------
static int32_t map_lookup(kvt_engine *e, const u32 *ids, u32 n_ctx, kvt_call_info *out, cudaStream_t s) {
  // plan: blocks, chunks, new key segments (all-or-nothing)
  u64 total_blocks = 0;
  for (u32 i = 0; i < n_ctx; ++i) total_blocks += e->ctxs[ids[i]].tok_len / 16;
  if (total_blocks > e->cfg.max_batch_blocks) return fail(e, KVT_E_NOSPACE, "batch exceeds max_batch_blocks");
  std::vector<int> newseg(n_ctx, -1);
  for (u32 i = 0; i < n_ctx; ++i) {
    u64 nb = e->ctxs[ids[i]].tok_len / 16;
    if (!nb) continue;
    newseg[i] = seg_new(e, nb);
    if (newseg[i] < 0 && e->dirty) {   // key lists that are only kept for the pending classification may be in the way
      int32_t rc = do_classify(e, s);
      if (rc) { for (u32 j = 0; j < i; ++j) seg_deref(e, newseg[j]); return rc; }
      newseg[i] = seg_new(e, nb);
    }
    if (newseg[i] < 0) {
      for (u32 j = 0; j < i; ++j) seg_deref(e, newseg[j]);
      return fail(e, KVT_E_NOSPACE, "key arena full");
    }
  }
  int32_t r = stage_acquire(e);
  if (r) { for (int sg : newseg) seg_deref(e, sg); return r; }
  // An error leaves the engine unchanged: the host-side changes below are made on the contexts themselves (the
  // kernels need the new layout), with copies kept aside; a failure puts the copies back and gives the new key
  // segments up. The old segments are only released once the call has succeeded. On the device, the kernels of a
  // failed call have written nothing but scratch and the new segments (k_lock_hits does nothing once the error
  // word is set).
  if (e->now == 0xFFFFFFFFu) { for (int sg : newseg) seg_deref(e, sg); return fail(e, KVT_E_NOSPACE, "logical clock exhausted"); }
  std::vector<Ctx> saved(n_ctx);
  for (u32 i = 0; i < n_ctx; ++i) saved[i] = e->ctxs[ids[i]];
  const u32 saved_now = e->now, saved_depth = e->max_depth;
  const bool saved_dirty = e->dirty;
  const u64 saved_rehashed = e->st.blocks_rehashed;
  auto rollback = [&](int32_t code) {
    for (u32 i = 0; i < n_ctx; ++i) e->ctxs[ids[i]] = std::move(saved[i]);
    for (int sg : newseg) seg_deref(e, sg);
    e->now = saved_now; e->max_depth = saved_depth; e->dirty = saved_dirty; e->st.blocks_rehashed = saved_rehashed;
    return code;
  };
#define CUR(call)                                                                                  \
  do {                                                                                             \
    cudaError_t _e = (call);                                                                       \
    if (_e != cudaSuccess) {                                                                       \
      e->err = std::string(#call) + ": " + cudaGetErrorString(_e);                                 \
      return rollback(KVT_E_CUDA);                                                                 \
    }                                                                                              \
  } while (0)
  e->now += 1;
  HashCtx *hd = reinterpret_cast<HashCtx *>(e->h_desc);
  std::vector<std::pair<u32, u32>> n_seq_chunks;   // per listed sequence: chunks in the all-blocks grid / in the digest grid
  std::vector<int> dev_idx(n_ctx, -1);
  u32 nd = 0, chunk_base = 0, dchunk_base = 0, blk_base = 0;
  bool long_seq = false;   // some sequence has so many chunks to digest that its carries come from the scan kernel
  u32 *h_hit = e->h_ctxres, *h_hbm = e->h_ctxres + e->cfg.max_contexts, *h_host = e->h_ctxres + 2 * e->cfg.max_contexts,
      *h_remote = e->h_ctxres + 3 * e->cfg.max_contexts;
  for (u32 i = 0; i < n_ctx; ++i) {
    Ctx &c = e->ctxs[ids[i]];
    for (Msg &m : c.msgs) if (m.state == MS_SUSPENDED) m.state = MS_ACTIVE;  // reactivation (Section 5.2)
    c.in_flight = true;
    c.map_dirty = true;
    c.mat_bounds.clear();
    u32 pos = 0;
    for (const Msg &m : c.msgs) { c.mat_bounds.push_back({pos, pos + m.len}); pos += m.len; }
    u32 nb = (u32)(c.tok_len / 16);
    // incremental hashing: the leading blocks this context still maps have unchanged tokens, so their keys
    // (and the chain carries kept per chunk) are taken over; hashing resumes at the last chunk boundary
    u32 first = 0;
    u64 old_key_off = 0, old_carry_off = 0;
    if (c.keyseg >= 0 && nb) {
      first = std::min(c.valid_blocks, nb) / CHUNK * CHUNK;
      old_key_off = e->segs[c.keyseg].off;
      old_carry_off = old_key_off + e->segs[c.keyseg].keycap;
    }
    c.keyseg = newseg[i];     // the old segment is released after the call has succeeded (it is read by this call's kernels)
    c.mat_blocks = c.valid_blocks = nb;
    e->max_depth = std::max(e->max_depth, nb);
    if (nb) {
      const KeySeg &sg = e->segs[c.keyseg];
      HashCtx d;
      d.tok_off = c.tok_off; d.key_off = sg.off; d.carry_off = sg.off + sg.keycap;
      d.old_key_off = old_key_off; d.old_carry_off = old_carry_off;
      d.n_blocks = nb; d.first = first; d.chunk_base = chunk_base; d.dchunk_base = dchunk_base; d.blk_base = blk_base; d.pad = 0;
      h_hit[nd] = nb; h_hbm[nd] = 0; h_host[nd] = 0; h_remote[nd] = 0;
      dev_idx[i] = (int)nd;
      hd[nd++] = d;
      chunk_base += cdiv(nb, CHUNK);
      dchunk_base += cdiv(nb - first, CHUNK);
      long_seq = long_seq || cdiv(nb - first, CHUNK) > FOLD_MAX_CHUNKS;
      n_seq_chunks.push_back({cdiv(nb, CHUNK), cdiv(nb - first, CHUNK)});
      blk_base += nb;
      e->st.blocks_rehashed += nb - first;
    }
  }
  e->dirty = true;
  if (nd) {
    u32 *d_res = e->dp<u32>(e->L.ctxres);
    const u32 C = e->cfg.max_contexts;
    // chunk -> sequence maps of the two grids, right behind the descriptors (one upload)
    u32 *h_map = reinterpret_cast<u32 *>(hd + nd), *h_dmap = h_map + chunk_base;
    {
      u32 k = 0, dk = 0;
      for (u32 q = 0; q < nd; ++q) {
        for (u32 j = 0; j < n_seq_chunks[q].first; ++j) h_map[k++] = q;
        for (u32 j = 0; j < n_seq_chunks[q].second; ++j) h_dmap[dk++] = q;
      }
    }
    TRACE(s, "begin");
    // one upload: zeroed status words, the per-context result words (prefix length = all blocks, no hits yet),
    // descriptors and chunk maps
    std::memset(e->h_status, 0, ST_WORDS * 4);
    {
      const u32 n16 = (u32)cdiv((e->L.desc - e->L.status) + nd * sizeof(HashCtx) + ((u64)chunk_base + dchunk_base) * 4, 16);
      KL(k_copy_words, std::min<u32>(cdiv(n16, 256), 64u), 256, s, (const uint4 *)e->h_status, (uint4 *)e->d_status, n16, e->copy_delay_ns);
    }
    HashArgs ha;
    ha.tokens = e->d_tokens; ha.keys = e->d_keys; ha.carry_base = e->d_keys; ha.ctx = e->dp<HashCtx>(e->L.desc); ha.n_ctx = nd;
    ha.agg = e->dp<u64>(e->L.agg); ha.h0 = e->h0; ha.single = HashCtx{}; ha.carries_ready = long_seq;
    ha.chunk_ctx = reinterpret_cast<const u32 *>(ha.ctx + nd); ha.dchunk_ctx = ha.chunk_ctx + chunk_base;
    LookupArgs la;
    la.tab = e->tab; la.b_ent = e->dp<u32>(e->L.s0); la.hit_len = d_res; la.status = e->d_status;
    LockArgs lk;
    lk.ent = e->ent; lk.b_ent = la.b_ent; lk.hit_len = d_res; lk.n_hbm = d_res + C; lk.n_host = d_res + 2 * C; lk.n_remote = d_res + 3 * C;
    lk.now = e->now; lk.status = e->d_status;
    if (e->profiling) CUR(cudaEventRecord(e->ev_h0, s));
    if (e->lookup_variant != 2) {
      const bool dg = dchunk_base != 0;
      TRACE(s, "uploads");
      if (dg) { launch_attr(e, false, true, k_hash_digest, dchunk_base, CHUNK, s, ha); e->st.kernel_launches++; }
      if (long_seq) KL(k_hash_carry, nd, 1024, s, ha);
      TRACE(s, "digest");
      // two keys per thread by default; one or four measured within 3 % of it: the probes of a cold table are bound
      // by the number of outstanding misses the memory system carries, not by what a thread issues
      if (e->lookup_variant == 3) launch_meta(e, true, k_hash_finish_lookup<1>, chunk_base, CHUNK, s, ha, la);
      else if (e->lookup_variant == 4) launch_meta(e, true, k_hash_finish_lookup<4>, chunk_base, CHUNK / 4, s, ha, la);
      else launch_meta(e, true, k_hash_finish_lookup<2>, chunk_base, CHUNK / 2, s, ha, la);
    } else {
      ChainState cs;
      cs.flags = e->dp<u32>(e->L.cflags); cs.ticket = cs.flags + chunk_base; cs.incl = e->dp<u64>(e->L.carry);
      cs.spin_limit = e->wait_limit;   // polls of (one L2 round trip + 40 ns): far beyond any real wait, still bounded
      CUR(cudaMemsetAsync(cs.flags, 0, (chunk_base + 1) * 4ull, s));
      KL(k_hash_lookup_fused, chunk_base, CHUNK, s, ha, la, cs);
    }
    TRACE(s, "finish");
    KLD(k_lock_hits<4>, chunk_base, CHUNK / 4, s, ha, lk);
    TRACE(s, "lock");
    if (e->profiling) CUR(cudaEventRecord(e->ev_h1, s));
    r = launch_ok(e);
    if (r) return rollback(r);
    // one read-back: status words and result words, written into the staging area by a kernel
    {
      const u32 n16 = (u32)cdiv((e->L.ctxres - e->L.status) + 4ull * C * 4, 16);
      launch_attr(e, false, true, k_copy_words, std::min<u32>(cdiv(n16, 256), 64u), 256, s, (const uint4 *)e->d_status, (uint4 *)e->h_status, n16, e->copy_delay_ns);
      e->st.kernel_launches++;
    }
    r = launch_ok(e);
    if (r) return rollback(r);
    CUR(cudaStreamSynchronize(s));
    TRACE(s, "results");
    if (e->profiling) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, e->ev_h0, e->ev_h1) == cudaSuccess) { e->st.lookup_ns += (u64)((double)ms * 1e6); e->st.lookup_blocks += blk_base; }
    }
    TRACE_DUMP("lookup");
    r = status_code(e);
    if (r) return rollback(r);
  }
#undef CUR
  for (u32 i = 0; i < n_ctx; ++i) seg_deref(e, saved[i].keyseg);
  for (u32 i = 0; i < n_ctx; ++i) {
    Ctx &c = e->ctxs[ids[i]];
    int k = dev_idx[i];
    c.hit_len = k >= 0 ? h_hit[k] : 0;
    c.n_hit_hbm = k >= 0 ? h_hbm[k] : 0;
    c.n_hit_host = k >= 0 ? h_host[k] : 0;
    c.n_hit_remote = k >= 0 ? h_remote[k] : 0;
    c.held = c.hit_len;
    if (e->cfg.policy_flags & KVT_POLICY_NO_LIFECYCLE) {   // nothing is known to be Temporary or Pinned
      c.n_admissible = c.mat_blocks - c.hit_len;
      c.n_pinned = 0;
    } else {
      c.n_admissible = first_temporary_block(c, c.hit_len, c.mat_blocks) - c.hit_len;
      c.n_pinned = count_pinned_blocks(c, c.hit_len, c.hit_len + c.n_admissible);
    }
    e->st.blocks_hashed += c.mat_blocks;
    e->st.hits_hbm += c.n_hit_hbm; e->st.hits_host += c.n_hit_host; e->st.hits_remote += c.n_hit_remote;
    e->st.misses += c.mat_blocks - c.hit_len;
    out[i] = kvt_call_info{c.mat_blocks, c.hit_len, c.n_hit_hbm, c.n_hit_host, c.n_admissible, 0, c.held, c.n_pinned, c.n_hit_remote};
  }
  return KVT_OK;
}

static int32_t map_admit(kvt_engine *e, const u32 *ids, u32 n_ctx, kvt_call_info *out, cudaStream_t s) {
  std::vector<u32> held0(n_ctx), cur(n_ctx), lim(n_ctx);
  std::vector<bool> stopped(n_ctx, false);
  for (u32 i = 0; i < n_ctx; ++i) {
    Ctx &c = e->ctxs[ids[i]];
    held0[i] = cur[i] = c.held;
    lim[i] = c.hit_len + c.n_admissible;
    if (cur[i] >= lim[i]) stopped[i] = true;
  }
  const u32 C = e->cfg.max_contexts;
  u32 first = 0;
  int32_t rc = KVT_OK;
  while (rc == KVT_OK) {
    while (first < n_ctx && stopped[first]) ++first;
    if (first == n_ctx) break;
    // claims may fill the table: keep live + tombstones + candidates below 3/4 of the capacity
    u64 cap = (u64)e->tab.mask + 1, used = (u64)e->occ[0] + e->occ[1] + e->occ[2] + e->tombs;
    if (used + 1 > cap * 3 / 4 || (e->tombs && used + e->cfg.max_batch_blocks > cap * 3 / 4)) {
      rc = table_rebuild(e, s);
      if (rc) break;
      used = (u64)e->occ[0] + e->occ[1] + e->occ[2];
    }
    u64 budget = std::min<u64>(cap * 3 / 4 - used, e->cfg.max_batch_blocks);
    rc = stage_acquire(e);
    if (rc) break;
    AdmitCtx *hd = reinterpret_cast<AdmitCtx *>(e->h_desc);
    u32 *h_stop = e->h_ctxres + 4 * C;
    u32 nd = 0, n_cand = 0;
    std::vector<u32> who;
    for (u32 i = first; i < n_ctx && n_cand < budget; ++i) {
      if (stopped[i]) continue;
      Ctx &c = e->ctxs[ids[i]];
      u32 take = (u32)std::min<u64>(lim[i] - cur[i], budget - n_cand);
      AdmitCtx d;
      d.key_off = e->segs[c.keyseg].off; d.cand_base = n_cand; d.b_start = cur[i]; d.b_end = cur[i] + take; d.res = nd;
      h_stop[nd] = d.b_end;
      hd[nd++] = d;
      who.push_back(i);
      n_cand += take;
      if (take < lim[i] - cur[i]) break;  // the rest of this context goes to the next round
    }
    u32 n_free = e->cfg.n_hbm_blocks - e->occ[0];
    AdmitArgs a;
    a.tab = e->tab; a.ent = e->ent; a.keys = e->d_keys; a.ctx = e->dp<AdmitCtx>(e->L.desc); a.n_ctx = nd; a.n_cand = n_cand;
    a.cslot = e->dp<u32>(e->L.s0); a.flag = e->dp<u32>(e->L.s1); a.aux = e->dp<u32>(e->L.s2); a.krank = e->dp<u32>(e->L.s3);
    a.freelist = e->dp<u32>(e->L.freelist); a.n_free = n_free; a.stop = e->dp<u32>(e->L.ctxres) + 4 * C;
    a.now = e->now; a.status = e->d_status;
    a.fresh = e->dp<u32>(e->L.fresh); a.fresh_base = e->n_fresh;
    if ((u64)e->n_fresh + n_free > e->ent.n_total) { rc = fail(e, KVT_E_DEVICE, "list of new entries would overflow"); break; }
    {   // descriptors and stop words up, status words zeroed: one small kernel
      std::memset(e->h_status, 0, ST_WORDS * 4);
      SegCopy up(e, s);
      up.add(e->dp<u8>(e->L.desc), hd, nd * sizeof(AdmitCtx));
      up.add(a.stop, h_stop, nd * 4ull);
      up.add(e->d_status, e->h_status, ST_WORDS * 4);
      up.flush();
    }
    u32 g = cdiv(n_cand, TPB);
    KLM(k_admit_claim, g, TPB, s, a);
    KLM(k_admit_resolve, g, TPB, s, a);
    rc = compact_indices(e, s, PredOwner{a.flag}, EmitRank{a.krank}, n_cand, ST_NEW);
    if (rc) break;
    rc = compact_indices(e, s, PredFree{e->ent.key, 0}, EmitFree{e->dp<u32>(e->L.freelist), (u32)e->L.LB}, e->cfg.n_hbm_blocks, ST_FREE);
    if (rc) break;
    KL(k_admit_stop, g, TPB, s, a);
    KLM(k_admit_apply, g, TPB, s, a);
    rc = launch_ok(e);
    if (rc) break;
    {
      SegCopy down(e, s);
      down.add(h_stop, a.stop, nd * 4ull);
      down.add(e->h_status, e->d_status, ST_WORDS * 4);
      down.flush();
    }
    rc = launch_ok(e);
    if (rc) break;
    CU(cudaStreamSynchronize(s));
    rc = status_code(e);
    if (rc) break;
    e->occ[0] += e->h_status[ST_INSERTED];
    e->n_fresh += e->h_status[ST_INSERTED];
    e->tombs += e->h_status[ST_TOMBS];
    e->st.inserted += e->h_status[ST_INSERTED];
    e->st.adopted += e->h_status[ST_ADOPTED];
    for (u32 k = 0; k < nd; ++k) {
      u32 i = who[k];
      const AdmitCtx &d = hd[k];
      cur[i] = h_stop[k];
      if (h_stop[k] < d.b_end || cur[i] >= lim[i]) stopped[i] = true;
    }
    e->dirty = true;
  }
  for (u32 i = 0; i < n_ctx; ++i) {
    Ctx &c = e->ctxs[ids[i]];
    c.held = cur[i];
    out[i] = kvt_call_info{c.mat_blocks, c.hit_len, c.n_hit_hbm, c.n_hit_host, c.n_admissible, cur[i] - held0[i], c.held, c.n_pinned,
                           c.n_hit_remote};
  }
  return rc;
}

int32_t kvt_map_blocks(kvt_engine *e, const uint32_t *ctx_ids, uint32_t n_ctx, uint32_t phase, kvt_call_info *out,
                       void *stream) {
  if (!e || !ctx_ids || !out || n_ctx == 0 || phase > 1) return KVT_E_INVAL;
  for (u32 i = 0; i < n_ctx; ++i)
    if (!get_ctx(e, ctx_ids[i])) return fail(e, KVT_E_NOCTX, "map_blocks: unknown context");
  {
    std::vector<u32> sorted(ctx_ids, ctx_ids + n_ctx);
    std::sort(sorted.begin(), sorted.end());
    if (std::adjacent_find(sorted.begin(), sorted.end()) != sorted.end()) return fail(e, KVT_E_INVAL, "map_blocks: duplicate context");
  }
  for (u32 i = 0; i < n_ctx; ++i) {
    bool f = e->ctxs[ctx_ids[i]].in_flight;
    if (phase == KVT_MAP_LOOKUP && f) return fail(e, KVT_E_STATE, "lookup: context already in flight");
    if (phase == KVT_MAP_ADMIT && !f) return fail(e, KVT_E_STATE, "admit: context not in flight");
  }
  cudaStream_t s = (cudaStream_t)stream;
  return phase == KVT_MAP_LOOKUP ? map_lookup(e, ctx_ids, n_ctx, out, s) : map_admit(e, ctx_ids, n_ctx, out, s);
}

int32_t kvt_get_block_map(kvt_engine *e, uint32_t ctx, uint64_t *keys, uint8_t *tier, uint32_t *slot, uint32_t cap,
                          uint32_t *n, void *stream) {
  if (!e || !n) return KVT_E_INVAL;
  Ctx *c = get_ctx(e, ctx, true);
  if (!c) return fail(e, KVT_E_NOCTX, "get_block_map: unknown context");
  cudaStream_t s = (cudaStream_t)stream;
  u32 nb = c->mat_blocks;
  *n = nb;
  if (cap < nb) return KVT_E_BUFSZ;
  if (!nb) return KVT_OK;
  if (nb > e->cfg.max_batch_blocks) return fail(e, KVT_E_NOSPACE, "context exceeds max_batch_blocks");
  const u64 *dk = e->d_keys + e->segs[c->keyseg].off;
  int32_t r = status_zero(e, s);
  if (r) return r;
  KL(k_block_map, cdiv(nb, TPB), TPB, s, e->tab, e->ent, dk, nb, e->dp<u8>(e->L.map_tier), e->dp<u32>(e->L.map_slot), e->d_status);
  LAUNCH_CHECK();
  // results go through pinned staging: one synchronisation for everything
  u64 *hk = (u64 *)e->h_out; u32 *hs = (u32 *)(e->h_out + nb * 8ull); u8 *ht = e->h_out + nb * 12ull;
  if (keys) CU(cudaMemcpyAsync(hk, dk, nb * 8ull, cudaMemcpyDeviceToHost, s));
  if (slot) CU(cudaMemcpyAsync(hs, e->dp<u32>(e->L.map_slot), nb * 4ull, cudaMemcpyDeviceToHost, s));
  if (tier) CU(cudaMemcpyAsync(ht, e->dp<u8>(e->L.map_tier), nb, cudaMemcpyDeviceToHost, s));
  r = status_fetch(e, s);
  if (r) return r;
  r = status_code(e);
  if (r) return r;
  if (keys) std::memcpy(keys, hk, nb * 8ull);
  if (slot) std::memcpy(slot, hs, nb * 4ull);
  if (tier) std::memcpy(tier, ht, nb);
  return KVT_OK;
}

// ---- stage 3 -----------------------------------------------------------------------------------------------
int32_t kvt_classify(kvt_engine *e, void *stream) {
  if (!e) return KVT_E_INVAL;
  return (e->dirty || e->classify_mode == 1) ? do_classify(e, (cudaStream_t)stream) : KVT_OK;
}

int32_t kvt_get_states(kvt_engine *e, uint32_t tier, uint8_t *state, uint32_t cap, void *stream) {
  if (!e || !state || tier > 2) return KVT_E_INVAL;
  u32 n = e->tier_slots(tier);
  if (cap < n) return KVT_E_BUFSZ;
  if (!n) return KVT_OK;
  cudaStream_t s = (cudaStream_t)stream;
  int32_t r = ensure_classified(e, s);
  if (r) return r;
  u8 *d_out = e->dp<u8>(e->L.out_states);
  KL(k_states_out, cdiv(n, TPB), TPB, s, e->ent, e->tier_e0(tier), n, d_out);
  LAUNCH_CHECK();
  CU(cudaMemcpyAsync(state, d_out, n, cudaMemcpyDeviceToHost, s));
  CU(cudaStreamSynchronize(s));
  return KVT_OK;
}

int32_t kvt_get_entries(kvt_engine *e, uint32_t tier, uint64_t *keys, uint32_t *stamp, uint32_t *depth,
                        uint32_t *inflight, uint32_t *link, uint32_t cap, void *stream) {
  if (!e || tier > 2) return KVT_E_INVAL;
  u32 n = e->tier_slots(tier), e0 = e->tier_e0(tier);
  if (cap < n) return KVT_E_BUFSZ;
  if (!n) return KVT_OK;
  cudaStream_t s = (cudaStream_t)stream;
  if (keys) CU(cudaMemcpyAsync(keys, e->ent.key + e0, n * 8ull, cudaMemcpyDeviceToHost, s));
  if (stamp) CU(cudaMemcpyAsync(stamp, e->ent.stamp + e0, n * 4ull, cudaMemcpyDeviceToHost, s));
  if (depth) CU(cudaMemcpyAsync(depth, e->ent.depth + e0, n * 4ull, cudaMemcpyDeviceToHost, s));
  if (inflight) CU(cudaMemcpyAsync(inflight, e->ent.infl + e0, n * 4ull, cudaMemcpyDeviceToHost, s));
  if (link) CU(cudaMemcpyAsync(link, e->ent.link + e0, n * 4ull, cudaMemcpyDeviceToHost, s));
  CU(cudaStreamSynchronize(s));
  if (link && tier == KVT_TIER_HBM)   // entry ids of host copies -> host slot numbers
    for (u32 i = 0; i < n; ++i) if (link[i] != ENT_NONE) link[i] -= e->cfg.n_hbm_blocks;
  return KVT_OK;
}

// ---- stage 4 -----------------------------------------------------------------------------------------------
// The address under which a kernel can write to `p`, or nullptr if `p` is ordinary pageable host memory.
static void *device_view(const void *p) {
  cudaPointerAttributes at{};
  if (!p || cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  if (at.type == cudaMemoryTypeHost || at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged) return at.devicePointer;
  return nullptr;
}

int32_t kvt_select_victims(kvt_engine *e, uint32_t tier, uint32_t n_req, uint32_t flags, uint32_t *slots_out,
                           uint8_t *states_out, uint32_t cap, uint32_t *n_out, void *stream) {
  if (!e || tier > 2 || flags > 1 || !n_out || (!slots_out && cap)) return KVT_E_INVAL;
  *n_out = 0;
  u32 n = e->tier_slots(tier);
  if (!n || !n_req) return KVT_OK;
  cudaStream_t s = (cudaStream_t)stream;
  int32_t r = ensure_classified(e, s);
  if (r) return r;
  int32_t rr = stage_acquire(e);
  if (rr) return rr;
  SelArgs &a = *e->h_sel;   // pinned staging: uploaded below, read by every kernel of the sequence
  a = SelArgs{};
  a.ent = e->ent; a.e0 = e->tier_e0(tier); a.n_slots = n; a.n_req = n_req; a.now = e->now;
  a.stamp_bits = bit_length(e->now); a.depth_bits = bit_length(e->max_depth);
  a.mru = e->cfg.suspended_order == KVT_ORDER_MRU; a.status = e->d_status;
  a.max_rank = (flags & KVT_SEL_INCLUDE_PINNED) ? 3 : 2;
  a.one_tier = (e->cfg.policy_flags & KVT_POLICY_NO_LIFECYCLE) ? 1 : 0;
  a.copy_bit = (tier == KVT_TIER_HOST && (e->cfg.policy_flags & KVT_POLICY_INCLUSIVE)) ? 1 : 0;
  const u32 key_bits = 2 + a.copy_bit + a.stamp_bits + a.depth_bits;
  if (key_bits > 63) return fail(e, KVT_E_INVAL, "select: stamps and depths this large do not fit the 63-bit victim key");
  // composite = (key << slot_bits) | slot, searched most significant digit first: 11 bits, then 13 at a time
  a.slot_bits = bit_length(n - 1);
  {
    u32 left = key_bits + a.slot_bits, lev = 0;
    do {   // the search needs no further level once a bin cannot hold more than SEL_SLACK composites (they are unique)
      const u32 w = std::min(left, lev == 0 ? SEL_W0 : SEL_WN);
      left -= w;
      a.lev_lo[lev] = (u8)left; a.lev_w[lev] = (u8)w;
      ++lev;
    } while (left && (1ull << left) > SEL_SLACK);
    a.n_levels = lev;
  }
  u64 *kA = e->dp<u64>(e->L.keyA), *kB = e->dp<u64>(e->L.keyB);
  u32 *vA = e->dp<u32>(e->L.valA), *vB = e->dp<u32>(e->L.valB), *counts = e->dp<u32>(e->L.rcounts);
  u32 *row_total = counts + (u64)RADIX_BINS * (e->L.Nt / SORT_TILE + 1);
  a.slot_key = e->dp<u64>(e->L.slot_key); a.hist = e->dp<u32>(e->L.sel_hist); a.state = e->dp<SelState>(e->L.sel_state);
  a.cta_count = e->dp<u32>(e->L.sel_cta);
  a.pair_key = kA; a.pair_val = vA;
  const u32 n_emit = std::min(n_req, n);
  const u32 m_max = (u32)std::min<u64>((u64)n_emit + SEL_SLACK, n);   // the gathered set never exceeds this
  a.n_emit = n_emit; a.rank_shift = a.stamp_bits + a.depth_bits;
  // the victim list is written by the last kernel straight into the pinned staging area (mapped into the device's
  // address space like every pinned allocation): no copy after the kernels, the list is there when the stream is
  // ... and when the caller's arrays are themselves memory a kernel can write (pinned host or device memory, large
  // enough for min(n_req, slots)), the list goes straight there and nothing is copied afterwards
  u32 *h_slots = (u32 *)e->h_out; u8 *h_states = e->h_out + n_emit * 4ull;
  a.slots_out = h_slots; a.states_out = h_states;
  bool direct = false;
  if (cap >= n_emit) {
    void *ds = device_view(slots_out), *dt = states_out ? device_view(states_out) : nullptr;
    if (ds && (dt || !states_out)) { direct = true; a.slots_out = (u32 *)ds; if (dt) a.states_out = (u8 *)dt; }
  }
  const SelArgs *d_args = e->dp<SelArgs>(e->L.sel_args);
  {   // argument record up, status words zeroed: one small kernel
    static_assert(sizeof(SelArgs) % 4 == 0, "argument record is copied in words");
    std::memset(e->h_status, 0, ST_WORDS * 4);
    SegCopy up(e, s);
    up.add((void *)d_args, &a, sizeof(SelArgs));
    up.add(e->d_status, e->h_status, ST_WORDS * 4);
    up.flush();
  }
  rr = stage_release(e, s);
  if (rr) return rr;
  const u32 n_levels = a.n_levels, n_pass = cdiv(key_bits, RADIX_BITS);
  // sort grids cover the bound of the gathered set rounded up to a power of two of tiles (few distinct graphs)
  u32 tiles = 1;
  while (tiles < cdiv(m_max, SORT_TILE)) tiles *= 2;
  const u32 g = cdiv(n, SEL_TILE);
  // The sequence below is short kernels with fixed grids and buffers whose arguments all live in device memory,
  // i.e. launch-bound: it is captured once per (tier, level count, pass count) into a CUDA graph on a private
  // stream and replayed on the caller's stream with one launch.
  auto enqueue = [&](cudaStream_t q, bool count) {
    if (count) TRACE(q, "start");
    cudaMemsetAsync(a.hist, 0, (u64)n_levels * SEL_BINS * 4, q);
    if (count) TRACE(q, "memset");
    // (dependent launches were tried for this chain and lose: with kernels of 3-10 us the programmatic completion
    // costs more than the tail overlap saves, 85 -> 135 us; the key kernel alone carries the L2 window)
    launch_attr(e, true, false, k_sel_keys, g, SEL_CTA, q, d_args);
    if (count) TRACE(q, "keys");
    for (u32 lev = 1; lev < n_levels; ++lev) { k_sel_level<<<g, SEL_CTA, 0, q>>>(d_args, lev); if (count) TRACE(q, "level"); }
    k_sel_count<<<g, SEL_CTA, 0, q>>>(d_args);
    if (count) TRACE(q, "count");
    k_sel_gather<<<g, SEL_CTA, 0, q>>>(d_args);
    if (count) TRACE(q, "gather");
    u64 *ka = kA, *kb = kB; u32 *va = vA, *vb = vB;
    for (u32 p = 0; p < n_pass; ++p) {
      k_radix_hist<<<tiles, 256, 0, q>>>(ka, e->d_status, RADIX_BITS * p, counts);
      if (count) TRACE(q, "hist");
      k_radix_scan<<<RADIX_BINS / 8, 256, 0, q>>>(counts, row_total, e->d_status);
      if (count) TRACE(q, "scan");
      k_radix_scatter<<<tiles, 256, 0, q>>>(ka, va, kb, vb, e->d_status, RADIX_BITS * p, counts, row_total);
      if (count) TRACE(q, "scatter");
      std::swap(ka, kb); std::swap(va, vb);
    }
    if (count) e->st.kernel_launches += 3ull + (n_levels - 1) + 3ull * n_pass;
  };
  // where the sorted pairs end up: the passes swap the two buffers
  const u64 *k_final = (n_pass & 1) ? kB : kA;
  const u32 *v_final = (n_pass & 1) ? vB : vA;
  if (e->profiling) CU(cudaEventRecord(e->ev_h0, s));
  {
    kvt_engine::SelGraph &gr = e->sel_graph[tier][(u64)n_levels << 48 | (u64)n_pass << 32 | tiles];
    if (e->use_graphs && !gr.exec) {
      cudaGraph_t graph = nullptr;
      bool ok = cudaStreamBeginCapture(e->capture_stream, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
      if (ok) {
        enqueue(e->capture_stream, false);
        ok = cudaStreamEndCapture(e->capture_stream, &graph) == cudaSuccess && graph;
      }
      if (ok) ok = cudaGraphInstantiate(&gr.exec, graph, 0) == cudaSuccess;
      if (graph) cudaGraphDestroy(graph);
      if (!ok) { cudaGetLastError(); gr.exec = nullptr; e->use_graphs = false; }   // fall back to plain launches
    }
    if (e->use_graphs && gr.exec) {
      CU(cudaGraphLaunch(gr.exec, s));
      e->st.kernel_launches += 3ull + (n_levels - 1) + 3ull * n_pass;
    } else {
      enqueue(s, true);
    }
  }
  if (e->profiling) CU(cudaEventRecord(e->ev_h1, s));   // selection and sort; the list's way to the host comes after
  KL(k_sel_emit, std::min<u32>(cdiv(n_emit, 1024), (u32)e->sm_count * 8), 256, s, d_args, k_final, v_final);
  { SegCopy down(e, s, true); down.add(e->h_status, e->d_status, ST_WORDS * 4); down.flush(); }   // status words beside the list
  LAUNCH_CHECK();
  CU(cudaStreamSynchronize(s));
  TRACE_DUMP("select");
  if (e->profiling) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, e->ev_h0, e->ev_h1) == cudaSuccess) { e->st.select_ns += (u64)((double)ms * 1e6); e->st.select_slots += n; }
  }
  r = status_code(e);
  if (r) return r;
  const u32 total = e->h_status[ST_TOTAL];   // candidates of the tier
  if (e->h_status[ST_M] != e->h_status[ST_AUX] || e->h_status[ST_M] > m_max || e->h_status[ST_M] < std::min(n_req, total))
    return fail(e, KVT_E_DEVICE, "selection: gathered set does not match its histogram");
  u32 k = std::min(n_req, total);
  *n_out = k;
  if (cap < k) return KVT_E_BUFSZ;
  if (k && !direct) {
    std::memcpy(slots_out, h_slots, k * 4ull);
    if (states_out) std::memcpy(states_out, h_states, k);
  }
  return KVT_OK;
}

// ---- stage 5 -----------------------------------------------------------------------------------------------
// Shared body of offload / reload / release.
struct ListMode { bool allow_inflight, drop_dead, drop_all, reject_shadow, clean_ok, keep_copy; };
struct ListCounts { u32 done = 0, copied = 0, dropped = 0, clean = 0; };

static int32_t list_op(kvt_engine *e, cudaStream_t s, u32 src_tier, u32 dst_tier, const u32 *slots, u32 n,
                       const ListMode &m, ListCounts *out) {
  *out = ListCounts();
  if (n == 0) return KVT_OK;
  if (n > e->L.LB) return fail(e, KVT_E_NOSPACE, "list longer than max_batch_blocks");
  int32_t r = stage_acquire(e);
  if (r) return r;
  // the mapping counts are brought up to date before any entry moves or goes away (the pending updates name entries)
  r = ensure_classified(e, s); if (r) return r; r = stage_acquire(e); if (r) return r;
  std::memcpy(e->h_ids, slots, n * 4ull);
  u32 *d_ids = e->dp<u32>(e->L.ids);
  CU(cudaMemcpyAsync(d_ids, e->h_ids, n * 4ull, cudaMemcpyHostToDevice, s));
  r = stage_release(e, s);
  if (r) return r;
  r = status_zero(e, s);
  if (r) return r;
  CU(cudaMemcpyAsync(e->d_status + ST_CUT, &n, 4, cudaMemcpyHostToDevice, s));  // pageable source: staged before return
  ListArgs a;
  a.tab = e->tab; a.ent = e->ent; a.ids = d_ids; a.n = n; a.e0 = e->tier_e0(src_tier); a.n_slots = e->tier_slots(src_tier);
  a.dst_e0 = e->tier_e0(dst_tier);
  a.live = e->dp<u32>(e->L.s1); a.lidx = e->dp<u32>(e->L.s2);
  a.freelist = e->dp<u32>(e->L.freelist); a.n_free = e->tier_slots(dst_tier) - e->occ[dst_tier];
  a.pair_src = e->dp<u32>(e->L.pair_src); a.pair_dst = e->dp<u32>(e->L.pair_dst);
  a.allow_inflight = m.allow_inflight; a.drop_dead = m.drop_dead; a.drop_all = m.drop_all;
  a.reject_shadow = m.reject_shadow; a.clean_ok = m.clean_ok; a.keep_copy = m.keep_copy; a.status = e->d_status;
  a.w_cut = ST_CUT; a.w_nlive = ST_NLIVE; a.w_ndrop = ST_NDROP; a.w_nclean = ST_NCLEAN; a.w_nshdrop = ST_NSHDROP;
  u32 g = cdiv(n, TPB);
  KL(k_list_validate, g, TPB, s, a);
  r = compact_indices(e, s, PredLive{a.live}, EmitLive{a.lidx, a.n_free, e->d_status + ST_CUT, nullptr}, n, ST_TOTAL);
  if (r) return r;
  if (!m.drop_all) {
    r = compact_indices(e, s, PredFree{e->ent.key, a.dst_e0}, EmitFree{e->dp<u32>(e->L.freelist), (u32)e->L.LB},
                        e->tier_slots(dst_tier), ST_FREE);
    if (r) return r;
  }
  KL(k_list_apply, g, TPB, s, a);
  KL(k_list_unmark, g, TPB, s, a);
  LAUNCH_CHECK();
  const bool staged = !m.drop_all && staged_applies(e, src_tier, dst_tier);
  const u32 n_pairs_max = std::min(n, a.n_free);
  u32 *h_psrc = (u32 *)e->h_out, *h_pdst = h_psrc + e->L.LB;
  if (!m.drop_all && !staged) {
    r = launch_mover(e, s, src_tier, a.pair_src, dst_tier, a.pair_dst, n_pairs_max, e->d_status + ST_NLIVE);
    if (r) return r;
  }
  if (staged && n_pairs_max) {   // the copy-engine transfers are issued from the host: it needs the planned pairs
    CU(cudaMemcpyAsync(h_psrc, a.pair_src, n_pairs_max * 4ull, cudaMemcpyDeviceToHost, s));
    CU(cudaMemcpyAsync(h_pdst, a.pair_dst, n_pairs_max * 4ull, cudaMemcpyDeviceToHost, s));
  }
  r = status_fetch(e, s);
  if (r) return r;
  r = status_code(e);
  if (r) return r;
  if (staged && e->h_status[ST_NLIVE]) {
    r = staged_move(e, s, src_tier, h_psrc, dst_tier, h_pdst, std::min(e->h_status[ST_NLIVE], n_pairs_max));
    if (r) return r;
    CU(cudaStreamSynchronize(s));
  }
  out->copied = e->h_status[ST_NLIVE];
  out->dropped = e->h_status[ST_NDROP];
  out->clean = e->h_status[ST_NCLEAN];
  out->done = out->copied + out->dropped + out->clean;
  mover_account(e, out->copied);
  // occupancy: listed blocks leave the source tier unless they stay behind as clean copies; copies that
  // belonged to dropped blocks free their host slots as well
  e->occ[src_tier] -= out->done - (m.keep_copy ? out->copied : 0);
  if (!m.drop_all) e->occ[dst_tier] += out->copied;
  e->occ[KVT_TIER_HOST] -= e->h_status[ST_NSHDROP];
  e->tombs += e->h_status[ST_TOMBS];
  e->st.dropped += out->dropped;
  if (out->dropped && (e->cfg.policy_flags & KVT_POLICY_ORPHANS_DEAD)) e->dirty = true;   // reachability changed
  r = maybe_rebuild(e, s);
  if (r) return r;
  return out->done < n ? KVT_E_NOSPACE : KVT_OK;
}

int32_t kvt_offload(kvt_engine *e, const uint32_t *hbm_slots, uint32_t n, uint32_t *n_done, uint32_t *n_dropped, void *stream) {
  if (!e || (!hbm_slots && n) || !n_done || !n_dropped) return KVT_E_INVAL;
  ListMode m{};
  m.drop_dead = !(e->cfg.policy_flags & KVT_POLICY_NO_LIFECYCLE);
  m.clean_ok = true;
  ListCounts c;
  int32_t r = list_op(e, (cudaStream_t)stream, KVT_TIER_HBM, KVT_TIER_HOST, hbm_slots, n, m, &c);
  *n_done = c.done; *n_dropped = c.dropped;
  e->st.offloaded += c.copied + c.clean;
  e->st.offloaded_clean += c.clean;
  e->st.bytes_d2h += c.copied * e->block_bytes;
  if (r == KVT_E_NOSPACE) e->err = "host tier full";
  return r;
}

int32_t kvt_reload(kvt_engine *e, const uint32_t *host_slots, uint32_t n, uint32_t *n_done, void *stream) {
  if (!e || (!host_slots && n) || !n_done) return KVT_E_INVAL;
  ListMode m{};
  m.allow_inflight = true;
  m.reject_shadow = true;
  m.keep_copy = e->cfg.policy_flags & KVT_POLICY_INCLUSIVE;
  ListCounts c;
  int32_t r = list_op(e, (cudaStream_t)stream, KVT_TIER_HOST, KVT_TIER_HBM, host_slots, n, m, &c);
  *n_done = c.done;
  e->st.reloaded += c.copied;
  e->st.bytes_h2d += c.copied * e->block_bytes;
  if (r == KVT_E_NOSPACE) e->err = "HBM tier full";
  return r;
}

int32_t kvt_move(kvt_engine *e, uint32_t src_tier, uint32_t dst_tier, const uint32_t *slots, uint32_t n, uint32_t *n_done,
                 uint32_t *n_dropped, void *stream) {
  if (!e || (!slots && n) || !n_done || !n_dropped) return KVT_E_INVAL;
  *n_done = *n_dropped = 0;
  if (src_tier == KVT_TIER_HBM && dst_tier == KVT_TIER_HOST) return kvt_offload(e, slots, n, n_done, n_dropped, stream);
  if (src_tier == KVT_TIER_HOST && dst_tier == KVT_TIER_HBM) return kvt_reload(e, slots, n, n_done, stream);
  const bool down = src_tier == KVT_TIER_HOST && dst_tier == KVT_TIER_REMOTE;
  const bool up = src_tier == KVT_TIER_REMOTE && (dst_tier == KVT_TIER_HOST || dst_tier == KVT_TIER_HBM);
  if (!down && !up) return KVT_E_INVAL;
  ListMode m{};
  m.reject_shadow = true;
  if (down) m.drop_dead = !(e->cfg.policy_flags & KVT_POLICY_NO_LIFECYCLE);
  else m.allow_inflight = true;
  ListCounts c;
  int32_t r = list_op(e, (cudaStream_t)stream, src_tier, dst_tier, slots, n, m, &c);
  *n_done = c.done; *n_dropped = c.dropped;
  if (down) e->st.demoted += c.copied; else e->st.promoted += c.copied;
  if (dst_tier == KVT_TIER_HBM) e->st.bytes_h2d += c.copied * e->block_bytes;
  if (r == KVT_E_NOSPACE) e->err = "destination tier full";
  return r;
}

int32_t kvt_exchange(kvt_engine *e, const uint32_t *hbm_slots_out, uint32_t n_out, const uint32_t *host_slots_in,
                     uint32_t n_in, uint32_t *n_out_done, uint32_t *n_dropped, uint32_t *n_in_done, void *stream) {
  if (!e || (!hbm_slots_out && n_out) || (!host_slots_in && n_in) || !n_out_done || !n_dropped || !n_in_done) return KVT_E_INVAL;
  *n_out_done = *n_dropped = *n_in_done = 0;
  cudaStream_t s = (cudaStream_t)stream;
  if (n_out == 0 && n_in == 0) return KVT_OK;
  if (n_out > e->L.LB || n_in > e->L.LB) return fail(e, KVT_E_NOSPACE, "list longer than max_batch_blocks");
  int32_t r = ensure_classified(e, s);
  if (r) return r;
  r = stage_acquire(e);
  if (r) return r;
  u32 *d_in = e->dp<u32>(e->L.ids), *d_out = e->dp<u32>(e->L.ids2);
  if (n_in) { std::memcpy(e->h_ids, host_slots_in, n_in * 4ull); CU(cudaMemcpyAsync(d_in, e->h_ids, n_in * 4ull, cudaMemcpyHostToDevice, s)); }
  if (n_out) { std::memcpy(e->h_ids2, hbm_slots_out, n_out * 4ull); CU(cudaMemcpyAsync(d_out, e->h_ids2, n_out * 4ull, cudaMemcpyHostToDevice, s)); }
  r = stage_release(e, s);
  if (r) return r;
  r = status_zero(e, s);
  if (r) return r;
  CU(cudaMemcpyAsync(e->d_status + ST_CUT, &n_in, 4, cudaMemcpyHostToDevice, s));
  CU(cudaMemcpyAsync(e->d_status + ST_B_CUT, &n_out, 4, cudaMemcpyHostToDevice, s));
  // list A: incoming (host -> HBM); list B: outgoing (HBM -> host). Both are validated against the state the call
  // finds; then the victims are planned and applied first, the reloads after them, so that the incoming blocks
  // take the lowest free HBM slots including those the victims leave: the result of kvt_offload + kvt_reload.
  ListArgs a{}, b{};
  a.tab = b.tab = e->tab; a.ent = b.ent = e->ent; a.status = b.status = e->d_status;
  a.ids = d_in; a.n = n_in; a.e0 = e->tier_e0(KVT_TIER_HOST); a.n_slots = e->cfg.n_host_blocks; a.dst_e0 = 0;
  a.live = e->dp<u32>(e->L.s1); a.lidx = e->dp<u32>(e->L.s2); a.freelist = e->dp<u32>(e->L.freelist);
  a.n_free = e->cfg.n_hbm_blocks;      // upper bound; the count after the victims have left is the device word ST_FREE
  a.pair_src = e->dp<u32>(e->L.pair_src); a.pair_dst = e->dp<u32>(e->L.pair_dst);
  a.allow_inflight = 1; a.reject_shadow = 1; a.keep_copy = (e->cfg.policy_flags & KVT_POLICY_INCLUSIVE) ? 1 : 0;
  a.w_cut = ST_CUT; a.w_nlive = ST_NLIVE; a.w_ndrop = ST_NDROP; a.w_nclean = ST_NCLEAN; a.w_nshdrop = ST_NSHDROP;
  b.ids = d_out; b.n = n_out; b.e0 = 0; b.n_slots = e->cfg.n_hbm_blocks; b.dst_e0 = e->tier_e0(KVT_TIER_HOST);
  b.live = e->dp<u32>(e->L.s3); b.lidx = e->dp<u32>(e->L.s0); b.freelist = e->dp<u32>(e->L.freelist2);
  b.n_free = e->cfg.n_host_blocks - e->occ[1];
  b.pair_src = e->dp<u32>(e->L.pair_src2); b.pair_dst = e->dp<u32>(e->L.pair_dst2);
  b.drop_dead = !(e->cfg.policy_flags & KVT_POLICY_NO_LIFECYCLE); b.clean_ok = 1;
  b.w_cut = ST_B_CUT; b.w_nlive = ST_B_NLIVE; b.w_ndrop = ST_B_NDROP; b.w_nclean = ST_B_NCLEAN; b.w_nshdrop = ST_B_NSHDROP;
  const u32 ga = cdiv(n_in, TPB), gb = cdiv(n_out, TPB);
  if (n_in) KL(k_list_validate, ga, TPB, s, a);
  if (n_out) KL(k_list_validate, gb, TPB, s, b);
  if (n_out) {   // victims: plan against the host slots that are free now, apply
    r = compact_indices(e, s, PredLive{b.live}, EmitLive{b.lidx, b.n_free, e->d_status + ST_B_CUT, nullptr}, n_out, ST_B_TOTAL);
    if (r) return r;
    if (e->cfg.n_host_blocks) {
      r = compact_indices(e, s, PredFree{e->ent.key, b.dst_e0}, EmitFree{e->dp<u32>(e->L.freelist2), (u32)e->L.LB}, e->cfg.n_host_blocks, ST_B_FREE);
      if (r) return r;
    }
    KL(k_list_apply, gb, TPB, s, b);
    KL(k_list_unmark, gb, TPB, s, b);
  }
  if (n_in) {    // reloads: the free HBM slots now include what the victims left
    r = compact_indices(e, s, PredFree{e->ent.key, 0}, EmitFree{e->dp<u32>(e->L.freelist), (u32)e->L.LB}, e->cfg.n_hbm_blocks, ST_FREE);
    if (r) return r;
    r = compact_indices(e, s, PredLive{a.live}, EmitLive{a.lidx, a.n_free, e->d_status + ST_CUT, e->d_status + ST_FREE}, n_in, ST_TOTAL);
    if (r) return r;
    KL(k_list_apply, ga, TPB, s, a);
    KL(k_list_unmark, ga, TPB, s, a);
  }
  LAUNCH_CHECK();
  const bool staged = staged_applies(e, KVT_TIER_HBM, KVT_TIER_HOST);
  if (staged) {   // copy engines, both directions: the transfers are issued from the host, which needs the planned pairs
    u32 *h_isrc = (u32 *)e->h_out, *h_idst = h_isrc + e->L.LB, *h_osrc = h_idst + e->L.LB, *h_odst = h_osrc + e->L.LB;
    const u32 n_out_max = std::min(n_out, b.n_free);
    if (n_in) {
      CU(cudaMemcpyAsync(h_isrc, a.pair_src, n_in * 4ull, cudaMemcpyDeviceToHost, s));
      CU(cudaMemcpyAsync(h_idst, a.pair_dst, n_in * 4ull, cudaMemcpyDeviceToHost, s));
    }
    if (n_out_max) {
      CU(cudaMemcpyAsync(h_osrc, b.pair_src, n_out_max * 4ull, cudaMemcpyDeviceToHost, s));
      CU(cudaMemcpyAsync(h_odst, b.pair_dst, n_out_max * 4ull, cudaMemcpyDeviceToHost, s));
    }
    r = status_fetch(e, s);
    if (r) return r;
    r = status_code(e);
    if (r) return r;
    const u32 ni = std::min(e->h_status[ST_NLIVE], n_in), no = std::min(e->h_status[ST_B_NLIVE], n_out_max);
    if (ni + no) {
      // the staging area is reused by the call below: keep the lists aside
      std::vector<u32> v_isrc(h_isrc, h_isrc + ni), v_idst(h_idst, h_idst + ni), v_osrc(h_osrc, h_osrc + no), v_odst(h_odst, h_odst + no);
      r = stage_acquire(e);
      if (r) return r;
      r = staged_exchange(e, s, ni, v_isrc.data(), v_idst.data(), no, v_osrc.data(), v_odst.data());
      if (r) return r;
      CU(cudaStreamSynchronize(s));
    }
  }
  // one mover launch for both directions
  if (!e->metadata_only && !staged) {
    MoveArgs ma{}, mb{};
    ma.src = pool_view(e, KVT_TIER_HOST); ma.dst = pool_view(e, KVT_TIER_HBM); ma.src_ids = a.pair_src; ma.dst_ids = a.pair_dst;
    ma.n_pairs = n_in; ma.n_pairs_dev = e->d_status + ST_NLIVE;
    mb.src = pool_view(e, KVT_TIER_HBM); mb.dst = pool_view(e, KVT_TIER_HOST); mb.src_ids = b.pair_src; mb.dst_ids = b.pair_dst;
    mb.n_pairs = std::min(n_out, b.n_free); mb.n_pairs_dev = e->d_status + ST_B_NLIVE;
    ma.n_chunks = mb.n_chunks = (u32)e->n_chunks; ma.chunk_bytes = mb.chunk_bytes = (u32)e->chunk_bytes; ma.status = mb.status = e->d_status;
    u64 items = ((u64)ma.n_pairs + mb.n_pairs) * e->n_chunks;
    if (items) {
      const bool timed = e->profiling;
      if (timed) CU(cudaEventRecord(e->ev_m0, s));
      const bool queues_fit = (u64)std::max(ma.n_pairs, mb.n_pairs) * e->n_chunks < (1ull << 32);   // 32-bit unit counters
      if (e->chunk_bytes % 4096 == 0 && queues_fit) {
        // which reload lands in a slot a victim leaves (scratch of the selection, idle during this call)
        u32 *vic_of = e->dp<u32>(e->L.out_slots), *dep = e->dp<u32>(e->L.valA), *taken = e->dp<u32>(e->L.valB);
        CU(cudaMemsetAsync(vic_of, 0xFF, (u64)e->cfg.n_hbm_blocks * 4, s));
        if (mb.n_pairs) KL(k_xchg_mark, cdiv(mb.n_pairs, TPB), TPB, s, mb.src_ids, mb.n_pairs_dev, mb.n_pairs, vic_of, taken);
        if (ma.n_pairs) KL(k_xchg_link, cdiv(ma.n_pairs, TPB), TPB, s, ma.dst_ids, ma.n_pairs_dev, ma.n_pairs, vic_of, dep, taken);
        u32 tpc = (u32)(e->chunk_bytes / 4096);
        const u32 xl = e->link_dirs(KVT_TIER_HBM, KVT_TIER_HOST) * 2;
        if (xl) {
          u32 grid = e->mover_grid((items + 31) / 32, xl);
          KL((k_move_exchange<8, 1024>), grid, 1024, s, ma, mb, tpc, dep, taken, e->d_status + ST_QA);
        } else {
          u32 grid = e->mover_grid((items + 7) / 8, xl);
          KL((k_move_exchange<8, 256>), grid, 256, s, ma, mb, tpc, dep, taken, e->d_status + ST_QA);
        }
      } else {   // chunk sizes the tile kernel cannot split: victims out, then reloads in (stream order)
        const u32 xl = e->link_dirs(KVT_TIER_HBM, KVT_TIER_HOST);
        u32 g1 = mb.n_pairs ? e->mover_grid((u64)mb.n_pairs * e->n_chunks, xl) * (xl && !e->mover_max_ctas ? 4 : 1) : 0;
        u32 g2 = ma.n_pairs ? e->mover_grid((u64)ma.n_pairs * e->n_chunks, xl) * (xl && !e->mover_max_ctas ? 4 : 1) : 0;
        if (g1) KL(k_move_blocks<4>, g1, 256, s, mb);
        if (g2) KL(k_move_blocks<4>, g2, 256, s, ma);
      }
      if (timed) { CU(cudaEventRecord(e->ev_m1, s)); e->mover_timed = true; }
      LAUNCH_CHECK();
    }
  }
  if (!staged) {
    r = status_fetch(e, s);
    if (r) return r;
    r = status_code(e);
    if (r) return r;
  }
  const u32 *h = e->h_status;
  const u32 in_copied = h[ST_NLIVE], out_copied = h[ST_B_NLIVE], out_drop = h[ST_B_NDROP], out_clean = h[ST_B_NCLEAN];
  mover_account(e, (u64)in_copied + out_copied);
  *n_in_done = in_copied;
  *n_out_done = out_copied + out_drop + out_clean;
  *n_dropped = out_drop;
  e->occ[KVT_TIER_HBM] += in_copied;
  if (!a.keep_copy) e->occ[KVT_TIER_HOST] -= in_copied;
  e->occ[KVT_TIER_HBM] -= *n_out_done;
  e->occ[KVT_TIER_HOST] += out_copied;
  e->occ[KVT_TIER_HOST] -= h[ST_B_NSHDROP];
  e->tombs += h[ST_TOMBS];
  e->st.dropped += out_drop;
  if (out_drop && (e->cfg.policy_flags & KVT_POLICY_ORPHANS_DEAD)) e->dirty = true;   // reachability changed
  e->st.reloaded += in_copied; e->st.bytes_h2d += in_copied * e->block_bytes;
  e->st.offloaded += out_copied + out_clean; e->st.offloaded_clean += out_clean; e->st.bytes_d2h += out_copied * e->block_bytes;
  r = maybe_rebuild(e, s);
  if (r) return r;
  if (*n_in_done < n_in || *n_out_done < n_out) return fail(e, KVT_E_NOSPACE, "exchange: a tier ran out of free slots");
  return KVT_OK;
}

int32_t kvt_release(kvt_engine *e, uint32_t tier, const uint32_t *slots, uint32_t n, void *stream) {
  if (!e || tier > 2 || (!slots && n)) return KVT_E_INVAL;
  ListMode m{};
  m.drop_all = true;
  ListCounts c;
  return list_op(e, (cudaStream_t)stream, tier, tier, slots, n, m, &c);
}

int32_t kvt_compact(kvt_engine *e, uint32_t tier, uint32_t *n_moved, void *stream) {
  if (!e || tier > 2 || !n_moved) return KVT_E_INVAL;
  *n_moved = 0;
  cudaStream_t s = (cudaStream_t)stream;
  u32 n = e->tier_slots(tier), e0 = e->tier_e0(tier), n_occ = e->occ[tier];
  if (!n || !n_occ || n_occ == n) return KVT_OK;
  int32_t r = ensure_classified(e, s);   // before entries move
  if (r) return r;
  r = status_zero(e, s);
  if (r) return r;
  u32 *src = e->dp<u32>(e->L.pair_src), *dst = e->dp<u32>(e->L.pair_dst);
  r = compact_indices(e, s, PredHole{e->ent.key, e0, n_occ}, EmitList{dst}, n, ST_AUX);
  if (r) return r;
  r = compact_indices(e, s, PredMover{e->ent.key, e0, n_occ}, EmitList{src}, n, ST_NMOVED);
  if (r) return r;
  u32 n_max = std::min(n_occ, n - n_occ);
  KL(k_compact_apply, cdiv(n_max, TPB), TPB, s, e->tab, e->ent, e0, src, dst, e->d_status);
  LAUNCH_CHECK();
  r = launch_mover(e, s, tier, src, tier, dst, n_max, e->d_status + ST_NMOVED);
  if (r) return r;
  r = status_fetch(e, s);
  if (r) return r;
  r = status_code(e);
  if (r) return r;
  if (e->h_status[ST_AUX] != e->h_status[ST_NMOVED]) return fail(e, KVT_E_DEVICE, "compaction plan mismatch");
  *n_moved = e->h_status[ST_NMOVED];
  mover_account(e, *n_moved);
  e->st.compacted += *n_moved;
  e->st.bytes_d2d += *n_moved * e->block_bytes;
  return KVT_OK;
}

int32_t kvt_copy_blocks(kvt_engine *e, uint32_t src_tier, const uint32_t *src, uint32_t dst_tier, const uint32_t *dst,
                        uint32_t n, uint32_t flags, void *stream) {
  if (!e || src_tier > 2 || dst_tier > 2 || ((!src || !dst) && n)) return KVT_E_INVAL;
  if (e->metadata_only) return fail(e, KVT_E_INVAL, "copy_blocks on a metadata-only engine");
  if (n == 0) return KVT_OK;
  if (n > e->L.LB) return fail(e, KVT_E_NOSPACE, "list longer than max_batch_blocks");
  cudaStream_t s = (cudaStream_t)stream;
  const u32 *ds = src, *dd = dst;
  if (!(flags & KVT_IDS_ON_DEVICE)) {
    int32_t r = stage_acquire(e);
    if (r) return r;
    std::memcpy(e->h_ids, src, n * 4ull);
    std::memcpy(e->h_ids2, dst, n * 4ull);
    CU(cudaMemcpyAsync(e->dp<u32>(e->L.ids), e->h_ids, n * 4ull, cudaMemcpyHostToDevice, s));
    CU(cudaMemcpyAsync(e->dp<u32>(e->L.ids2), e->h_ids2, n * 4ull, cudaMemcpyHostToDevice, s));
    r = stage_release(e, s);
    if (r) return r;
    ds = e->dp<u32>(e->L.ids); dd = e->dp<u32>(e->L.ids2);
  }
  return launch_mover(e, s, src_tier, ds, dst_tier, dd, n, nullptr);
}

// ---- stand-alone hasher -----------------------------------------------------------------------------------
uint64_t kvt_hash_scratch_bytes(uint64_t n_tokens) {
  u64 n_chunks = (n_tokens / 16 + CHUNK - 1) / CHUNK;
  return (2 * std::max<u64>(n_chunks, 1) + 1) * 8;   // chunk aggregates, then chunk carries plus the final value
}

int32_t kvt_hash_tokens(const uint32_t *d_tokens, uint64_t n_tokens, uint64_t hash_seed, uint64_t *d_keys, void *d_scratch,
                        uint64_t scratch_bytes, void *stream) {
  u64 nb = n_tokens / 16;
  if (nb == 0) return KVT_OK;
  if (!d_tokens || !d_keys || !d_scratch || ((uintptr_t)d_tokens & 15) || ((uintptr_t)d_scratch & 7)) return KVT_E_INVAL;
  if (nb >= 0xFFFFFFFFull || scratch_bytes < kvt_hash_scratch_bytes(n_tokens)) return KVT_E_INVAL;
  cudaStream_t s = (cudaStream_t)stream;
  u32 n_chunks = cdiv(nb, CHUNK);
  HashArgs ha;
  ha.tokens = d_tokens; ha.keys = d_keys; ha.ctx = nullptr; ha.n_ctx = 1; ha.chunk_ctx = ha.dchunk_ctx = nullptr;
  ha.single = HashCtx{};
  ha.single.n_blocks = (u32)nb;
  ha.agg = (u64 *)d_scratch; ha.carry_base = (u64 *)d_scratch + n_chunks; ha.h0 = hash_h0(hash_seed);
  LookupArgs la{};
  ha.carries_ready = n_chunks > FOLD_MAX_CHUNKS;   // a long sequence: its chunk carries come from the scan kernel
  k_hash_digest<<<n_chunks, CHUNK, 0, s>>>(ha);
  if (ha.carries_ready) k_hash_carry<<<1, 1024, 0, s>>>(ha);
  k_hash_finish_lookup<1><<<n_chunks, CHUNK, 0, s>>>(ha, la);
  return cudaGetLastError() == cudaSuccess ? KVT_OK : KVT_E_CUDA;
}

// ---- hasher without allocation ------------------------------------------------------------------------------
// Scratch of the no-allocation hasher: chunk aggregates followed by chunk carries. File-scope device
// memory: in host code this name is only a handle, so its device address is queried below (with the
// caller's device current) and that pointer is what the kernels get.
constexpr u64 NOALLOC_MAX_CHUNKS = KVT_HASH_NOALLOC_MAX_TOKENS / 16 / CHUNK;
static __device__ __align__(256) unsigned long long g_noalloc_scratch[2 * NOALLOC_MAX_CHUNKS + 1];

int32_t kvt_hash_tokens_noalloc(const uint32_t *d_tokens, uint64_t n_tokens, uint64_t hash_seed, uint64_t *d_keys,
                                void *stream) {
  if (n_tokens > KVT_HASH_NOALLOC_MAX_TOKENS) return KVT_E_NOSPACE;   // beyond the built-in scratch
  u64 nb = n_tokens / 16;
  if (nb == 0) return KVT_OK;
  if (!d_tokens || !d_keys || ((uintptr_t)d_tokens & 15)) return KVT_E_INVAL;
  // The array's address on the current device. Asked for on every call: after the first call on a device (which
  // makes the runtime load this module there) it is a look-up, and nothing cached here can go stale when a device's
  // context is reset or be raced for by two host threads.
  void *sym = nullptr;
  if (cudaGetSymbolAddress(&sym, g_noalloc_scratch) != cudaSuccess || !sym) return KVT_E_CUDA;
  u64 *const scratch = (u64 *)sym;
  cudaStream_t s = (cudaStream_t)stream;
  u32 n_chunks = cdiv(nb, CHUNK);
  HashArgs ha;
  ha.tokens = d_tokens; ha.keys = d_keys; ha.ctx = nullptr; ha.n_ctx = 1; ha.chunk_ctx = ha.dchunk_ctx = nullptr;
  ha.single = HashCtx{};
  ha.single.n_blocks = (u32)nb;
  ha.agg = scratch; ha.carry_base = scratch + NOALLOC_MAX_CHUNKS; ha.h0 = hash_h0(hash_seed);
  LookupArgs la{};
  ha.carries_ready = n_chunks > FOLD_MAX_CHUNKS;   // a long sequence: its chunk carries come from the scan kernel
  k_hash_digest<<<n_chunks, CHUNK, 0, s>>>(ha);
  if (ha.carries_ready) k_hash_carry<<<1, 1024, 0, s>>>(ha);
  k_hash_finish_lookup<1><<<n_chunks, CHUNK, 0, s>>>(ha, la);
  return cudaGetLastError() == cudaSuccess ? KVT_OK : KVT_E_CUDA;
}

// ---- debug loader -------------------------------------------------------------------------------------------
int32_t kvt_debug_load_resident(kvt_engine *e, const uint64_t *keys, const uint8_t *state, const uint32_t *stamp,
                                const uint32_t *depth, const uint32_t *slot, uint32_t tier, uint32_t n, void *stream) {
  if (!e || tier > 2 || ((!keys || !state || !stamp || !depth || !slot) && n)) return KVT_E_INVAL;
  if (n == 0) return KVT_OK;
  u32 ns = e->tier_slots(tier);
  if (n > ns || n > e->L.LB) return fail(e, KVT_E_INVAL, "more blocks than slots");
  u32 max_stamp = 0, max_d = 0;
  {
    std::vector<u64> ks(keys, keys + n);
    std::vector<u32> ss(slot, slot + n);
    std::sort(ks.begin(), ks.end());
    std::sort(ss.begin(), ss.end());
    if (ks[0] < 2 || std::adjacent_find(ks.begin(), ks.end()) != ks.end() ||
        std::adjacent_find(ss.begin(), ss.end()) != ss.end() || ss.back() >= ns)
      return fail(e, KVT_E_INVAL, "bad keys or slots");
    for (u32 i = 0; i < n; ++i) {
      if (state[i] > 3) return fail(e, KVT_E_INVAL, "bad state");
      max_stamp = std::max(max_stamp, stamp[i]); max_d = std::max(max_d, depth[i]);
    }
  }
  if ((u64)e->occ[0] + e->occ[1] + e->occ[2] + e->tombs + n > ((u64)e->tab.mask + 1) * 3 / 4) return fail(e, KVT_E_NOSPACE, "table too full");
  // the victim key packs rank, recency and depth into 63 bits: stamps and depths that would not fit are refused here
  if (3 + bit_length(std::max(e->now, max_stamp)) + bit_length(std::max(e->max_depth, max_d)) > 63)
    return fail(e, KVT_E_INVAL, "stamp and depth too large for the victim key");
  cudaStream_t s = (cudaStream_t)stream;
  // stage the arrays in scratch: keys -> keyA, state -> out_states, stamp/depth/slot -> s1/s2/s3
  u64 *dk = e->dp<u64>(e->L.keyA);
  u8 *dst_state = e->dp<u8>(e->L.out_states);
  u32 *dsp = e->dp<u32>(e->L.s1), *ddp = e->dp<u32>(e->L.s2), *dsl = e->dp<u32>(e->L.s3);
  CU(cudaMemcpyAsync(dk, keys, n * 8ull, cudaMemcpyHostToDevice, s));
  CU(cudaMemcpyAsync(dst_state, state, n, cudaMemcpyHostToDevice, s));
  CU(cudaMemcpyAsync(dsp, stamp, n * 4ull, cudaMemcpyHostToDevice, s));
  CU(cudaMemcpyAsync(ddp, depth, n * 4ull, cudaMemcpyHostToDevice, s));
  CU(cudaMemcpyAsync(dsl, slot, n * 4ull, cudaMemcpyHostToDevice, s));
  int32_t r = status_zero(e, s);
  if (r) return r;
  LoadArgs a;
  a.tab = e->tab; a.ent = e->ent; a.keys = dk; a.state = dst_state; a.stamp = dsp; a.depth = ddp; a.slot = dsl;
  a.n = n; a.e0 = e->tier_e0(tier); a.n_slots = ns; a.status = e->d_status;
  KL(k_load_check, cdiv(n, TPB), TPB, s, a);
  KL(k_load_apply, cdiv(n, TPB), TPB, s, a);
  LAUNCH_CHECK();
  r = status_fetch(e, s);
  if (r) return r;
  r = status_code(e);
  if (r) return r;
  e->occ[tier] += n;
  for (const Ctx &c : e->ctxs) if (c.live) { e->full_dirty = e->dirty = true; break; }   // existing contexts may map the new keys
  e->now = std::max(e->now, max_stamp);
  e->max_depth = std::max(e->max_depth, max_d);
  return KVT_OK;
}

}  // extern "C"
