/*
 * kvt.h — C ABI of the lifecycle-aware KV cache engine hot path (GPU library libkvt.so).
 *
 * The library implements, for one GPU, the data-parallel part of a lifecycle-aware KV cache
 * manager for ReAct agents:
 *   (1) chained 16-token block hashing of agent contexts built by message-level primitives
 *       (Section 4.1, Table 3: append / replace / remove / fork / spawn / one_off),
 *   (2) lookup of those hashes in a GPU-resident open-addressing block table (reusable prefix),
 *   (3) derivation of each resident block's KV-level lifecycle state from message-level states
 *       (Section 5.2 state machine; Section 6.1, the paragraph on KV shared between contexts),
 *   (4) state-prioritised, recency-ordered victim selection (Algorithm 1; Section 6.2), and
 *   (5) movement of paged KV blocks between the HBM pool, a pinned host tier and an optional third tier (Section 7).
 *
 * General conventions
 *   - Plain C, no exceptions, no stdout. Every function returns an int32_t status: KVT_OK (0) or a
 *     negative KVT_E_* code. Unless a call documents partial progress through an out-count, a call
 *     that returns an error leaves the engine state unchanged.
 *   - Memory ownership: the caller allocates the HBM pool, the host pool (pinned, device-mapped
 *     memory), the device metadata arena and the device token arena, and passes raw pointers and
 *     byte sizes in kvt_config. The library never allocates or frees device memory and never frees
 *     caller memory. It does allocate a few MB of pinned HOST staging memory of its own in
 *     kvt_create and frees it in kvt_destroy.
 *   - "device pointer" = memory the GPU can dereference (cudaMalloc'd, or pinned mapped host
 *     memory under unified addressing). "host pointer" = ordinary host memory read/written by the
 *     CPU inside the call; it may be reused as soon as the call returns.
 *   - stream: a cudaStream_t passed as void*. All device work of a call is enqueued on it. Calls
 *     that return counts or data to the host synchronise that stream before returning (stated per
 *     call); kvt_copy_blocks is asynchronous.
 *   - An engine is not thread-safe; calls on one engine must be serialised by the caller and must
 *     all use streams that are ordered with respect to each other.
 *   - Every device-side loop (table probe loops) has an iteration cap; on overrun the kernel sets
 *     a device error word and returns normally, and the call reports KVT_E_DEVICE.
 *   - The library has no CPU fallback: without a usable CUDA device kvt_create fails with
 *     KVT_E_CUDA.
 */
#ifndef KVT_H_
#define KVT_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KVT_ABI_VERSION 3u
#define KVT_BLOCK_TOKENS 16u

/* ---- status codes -------------------------------------------------------------------------- */
#define KVT_OK          0
#define KVT_E_INVAL    -1  /* malformed argument (NULL pointer, bad enum, id in use, duplicate id) */
#define KVT_E_NOCTX    -2  /* unknown or terminated context */
#define KVT_E_RANGE    -3  /* message range or slot id out of bounds */
#define KVT_E_STATE    -4  /* op not allowed in the current state (in-flight context / in-flight block) */
#define KVT_E_NOSPACE  -5  /* a tier, the table or an arena is full; see the call's out-counts */
#define KVT_E_BUFSZ    -6  /* caller-provided output buffer too small */
#define KVT_E_DEVICE   -7  /* device error word set (probe cap exceeded, corrupt metadata) */
#define KVT_E_CUDA     -8  /* a CUDA runtime call failed; text via kvt_last_error */

/* ---- enums --------------------------------------------------------------------------------- */
/* Tiers (Section 7: a multi-tier engine spanning GPU HBM, host memory and remote memory). */
#define KVT_TIER_HBM   0u
#define KVT_TIER_HOST  1u
#define KVT_TIER_REMOTE 2u  /* third level of Section 7's hierarchy (remote memory); here one more caller-provided
                              device-accessible buffer stands in for it: cross-node transport is out of scope */
#define KVT_TIER_NONE  0xFFu   /* "not resident" in block maps */

/* HBM pool layouts. The host pool is always block-major. */
#define KVT_LAYOUT_LAYER_MAJOR 0u  /* chunk (layer l, kv) of slot s at ((l*2+kv)*n_hbm_blocks + s)*chunk_bytes */
#define KVT_LAYOUT_BLOCK_MAJOR 1u  /* slot s at s*block_bytes, chunk c at + c*chunk_bytes */

/* Recency direction inside the Suspended (live-but-idle) tier (Section 6.2 and the "w/o RO"
 * ablation of Section 8.3). */
#define KVT_ORDER_MRU 0u   /* most recently suspended first (the paper's policy, default) */
#define KVT_ORDER_LRU 1u   /* oldest first */

/* kvt_config.policy_flags */
#define KVT_POLICY_NO_LIFECYCLE 1u  /* the "w/o LT" ablation of Section 8.3: no lifecycle information reaches the
                                       policy. Every resident block is one tier ordered by suspended_order alone,
                                       offload copies every victim (nothing is known to be dead) and nothing bypasses
                                       admission. kvt_get_states still reports the true states (for metrics). */

#define KVT_POLICY_INCLUSIVE 2u     /* inclusive tiers (Section 7: a tier may retain a fast copy): kvt_reload leaves the
                                       block's bytes in its host slot as a clean copy linked to the HBM block; a later
                                       kvt_offload of that block hands it back to the copy without moving a byte.
                                       Copies occupy host slots, are the first victims of the host tier (state
                                       KVT_STATE_COPY), can be released on their own, and go away with their block. */
#define KVT_POLICY_ORPHANS_DEAD 4u   /* reachability-aware classification. A lookup reuses a contiguous prefix of a
                                       context's chain (Section 2.1: prefix-dependent validity), so a resident block
                                       behind a block that is no longer resident in any tier can never be hit again
                                       through that context. With this flag a context's mappings stop counting at
                                       its first non-resident block; a block that no context reaches any more
                                       classifies as dead, becomes a first victim and is dropped, not copied. The
                                       paper is silent on such orphans; without the flag they keep their state. */

/* Primitives and runtime events (Table 3; Section 5.2 "Runtime transitions"). */
#define KVT_OP_SPAWN         1u  /* register an independent, empty context */
#define KVT_OP_FORK          2u  /* register child `ctx` sharing messages [0, msg_end) of `parent` */
#define KVT_OP_APPEND        3u  /* append one message (tokens) */
#define KVT_OP_REPLACE       4u  /* replace messages [msg_start, msg_end) by one message (tokens) */
#define KVT_OP_REMOVE        5u  /* remove messages [msg_start, msg_end) */
#define KVT_OP_ONE_OFF       6u  /* mark the context (msg_start=0, msg_end=UINT32_MAX) or messages
                                    [msg_start, msg_end) for one inference (Temporary) */
#define KVT_OP_PREFILL_DONE  7u  /* prefill of the context's in-flight call completed */
#define KVT_OP_TERMINATE     8u  /* the context ends */
#define KVT_OP_PIN           9u  /* declare long-term retention of messages [msg_start, msg_end) */
#define KVT_OP_UNPIN        10u  /* release that protection */

/* kvt_op.flags */
#define KVT_OPF_TOKENS_ON_DEVICE 1u  /* op.tokens is a device pointer (device-to-device copy) */

/* kvt_map_blocks phases */
#define KVT_MAP_LOOKUP 0u
#define KVT_MAP_ADMIT  1u

/* kvt_select_victims flags */
#define KVT_SEL_INCLUDE_PINNED 1u  /* the incoming KV is Pinned: Pinned residents compete too (Algorithm 1, last branch) */

/* kvt_copy_blocks flags */
#define KVT_IDS_ON_DEVICE 1u  /* src/dst id arrays are device pointers */

/* KV-level lifecycle ranks reported by kvt_get_states / kvt_select_victims. They follow the
 * release order of Algorithm 1: Discarded (Expired or Temporary) < Suspended < Active < Pinned. */
#define KVT_STATE_DEAD    0u   /* no live message version maps the block */
#define KVT_STATE_IDLE    1u   /* live but idle: best mapped message state is Suspended */
#define KVT_STATE_ACTIVE  2u   /* live and active */
#define KVT_STATE_PINNED  3u   /* explicitly retained: competes for space only with incoming Pinned KV */
#define KVT_STATE_FREE    0xFFu /* slot holds no block */
#define KVT_STATE_COPY    0xFEu /* host slot holding only the clean copy of a block whose home is HBM (inclusive tiers) */
#define KVT_STATE_HAS_COPY 0x80u /* or-ed into the rank of an HBM victim that still has a clean host copy */

typedef struct kvt_engine kvt_engine;

/* ---- configuration -------------------------------------------------------------------------- */
typedef struct kvt_config {
  uint32_t abi_version;      /* KVT_ABI_VERSION */
  uint32_t block_tokens;     /* must be 16 */
  uint32_t n_layers;         /* KV geometry: a token's KV is n_layers * 2 (K,V) * n_kv_heads * head_dim * elem_bytes */
  uint32_t n_kv_heads;
  uint32_t head_dim;
  uint32_t elem_bytes;       /* 2 for bf16 */
  uint32_t pool_layout;      /* KVT_LAYOUT_* of the HBM pool */
  uint32_t n_hbm_blocks;     /* slots in the HBM tier (>= 1) */
  uint32_t n_host_blocks;    /* slots in the host tier (may be 0) */
  uint32_t table_capacity;   /* power of two, >= 2 * (n_hbm_blocks + n_host_blocks + n_remote_blocks) */
  uint32_t max_contexts;     /* context ids are 0 .. max_contexts-1 */
  uint32_t max_messages;     /* upper bound on messages with materialised positions, all contexts together */
  uint32_t max_batch_blocks; /* upper bound on the blocks hashed by one kvt_map_blocks call and on n of one list call */
  uint32_t policy_flags;     /* KVT_POLICY_* (0 = the paper's policy) */
  uint64_t max_tokens;       /* capacity of the device token arena, in tokens */
  uint64_t max_key_blocks;   /* capacity of the per-context key lists, in blocks (all contexts together) */
  uint64_t hash_seed;        /* seed of the block hash */
  uint32_t suspended_order;  /* KVT_ORDER_* */
  uint32_t n_remote_blocks;  /* slots in the remote tier (may be 0) */
  void *hbm_pool;  uint64_t hbm_pool_bytes;   /* device; NULL/0 = metadata-only engine (no payload is moved) */
  void *host_pool; uint64_t host_pool_bytes;  /* device-accessible pinned host memory; NULL/0 if metadata-only */
  void *dev_meta;  uint64_t dev_meta_bytes;   /* device metadata + scratch arena, 256-byte aligned */
  void *dev_tokens; uint64_t dev_tokens_bytes;/* device token arena, 256-byte aligned */
  void *remote_pool; uint64_t remote_pool_bytes; /* device-accessible memory of the remote tier; NULL/0 if none or metadata-only */
  void *stage_buf; uint64_t stage_bytes;         /* optional device memory (16-byte aligned; 64-512 MiB is plenty) for moves
                                                    between device memory and a pool in host memory: the mover kernel
                                                    gathers / scatters whole blocks through it and the copy engines carry
                                                    them over the link in large transfers, on two streams the library
                                                    creates, one per direction. NULL/0: the kernel reads / writes host
                                                    memory directly. Used for blocks of at least 512 KiB. */
} kvt_config;

/* Computes the byte sizes the caller must allocate for dev_meta and dev_tokens from the other
 * fields of cfg (pointer fields are ignored). Host-only. */
int32_t kvt_query_sizes(const kvt_config *cfg, uint64_t *meta_bytes, uint64_t *token_bytes);

/* Creates an engine on the current CUDA device. Validates cfg (KVT_E_INVAL), zero-initialises
 * the metadata arena on `stream` and synchronises it. The pools are not touched. */
int32_t kvt_create(const kvt_config *cfg, void *stream, kvt_engine **out);
int32_t kvt_destroy(kvt_engine *e);

/* ---- stage 0: message-level primitives (Table 3; Section 5.1; Section 5.2) ------------------ */
typedef struct kvt_op {
  uint32_t op;          /* KVT_OP_* */
  uint32_t ctx;         /* context the op applies to (FORK: the new child) */
  uint32_t parent;      /* FORK only */
  uint32_t msg_start;   /* REPLACE / REMOVE / ONE_OFF: first message of the range */
  uint32_t msg_end;     /* one past the last message; FORK: number of inherited messages */
  uint32_t n_tokens;    /* APPEND / REPLACE: length of the new message (may be 0) */
  uint32_t flags;       /* KVT_OPF_* */
  uint32_t reserved;    /* must be 0 */
  const uint32_t *tokens; /* APPEND / REPLACE payload: host pointer (pageable memory is copied before return;
                             pinned memory must stay unchanged until the stream has passed the call) or
                             device pointer with KVT_OPF_TOKENS_ON_DEVICE */
} kvt_op;

/* Applies one primitive or runtime event to a context, strictly in program order per context
 * (Section 5.1). Host bookkeeping plus, for token-carrying ops, a copy of the tokens into the
 * device token arena and, for PREFILL_DONE / TERMINATE of an in-flight context, one kernel that
 * releases the in-flight locks of the blocks the context holds.
 *   APPEND: new message is Active, or Temporary if the context is one_off. No KV effect until the
 *     next call (KV-existence gating, Section 5.1).
 *   REPLACE / REMOVE at message s: the old versions of s and of every later message expire for
 *     this context only: the context stops mapping every block from the block containing the first
 *     token of message s on (prefix-dependent validity, Section 5.1). Requires s < e <= #messages.
 *   FORK: the child gets Active copies of parent messages [0, msg_end) and immediately maps the
 *     still-valid blocks they cover; parent and child evolve independently afterwards.
 *   ONE_OFF: listed (or all current and future) messages become Temporary.
 *   PREFILL_DONE: Active -> Suspended; advances the logical clock; stamps and unlocks held blocks.
 *   PIN / UNPIN: listed messages become Pinned / Pinned ones return to Suspended (Temporary in a one_off
 *     context). Pinned messages are not touched by call begin, PREFILL_DONE or the whole-context ONE_OFF.
 *   TERMINATE: ordinary messages expire. Without Pinned messages the context stops mapping anything and
 *     its id becomes free; with Pinned messages it is kept (they retain their protection), accepts only
 *     UNPIN (which then expires them), and goes away with its last Pinned message.
 * Errors: KVT_E_NOCTX unknown context; KVT_E_INVAL id in use / bad op / NULL tokens;
 * KVT_E_RANGE bad message range; KVT_E_STATE edit or fork-from of an in-flight context, or
 * PREFILL_DONE of a context that is not in flight; KVT_E_NOSPACE token arena full.
 * Does not synchronise the stream. */
int32_t kvt_apply_op(kvt_engine *e, const kvt_op *op, void *stream);

/* ---- stages 1+2 (+ admission): hash, lookup, admit ------------------------------------------- */
typedef struct kvt_call_info {
  uint32_t n_blocks;      /* full 16-token blocks of the context's token sequence */
  uint32_t hit_len;       /* leading blocks found resident at LOOKUP (the reusable prefix) */
  uint32_t n_hit_hbm;     /* of those, resident in HBM */
  uint32_t n_hit_host;    /* of those, resident in the host tier (reload them before use) */
  uint32_t n_admissible;  /* blocks after the prefix that may enter reusable storage (Temporary bypass) */
  uint32_t n_admitted;    /* ADMIT: blocks this call newly holds (inserted or adopted) */
  uint32_t n_held;        /* leading blocks locked in flight for this context after the call */
  uint32_t n_pinned;      /* of the admissible blocks, those touched by a Pinned message */
  uint32_t n_hit_remote;  /* of the reusable prefix, blocks resident in the remote tier (kvt_move them up before use) */
} kvt_call_info;

/* phase KVT_MAP_LOOKUP — one LLM call begins for each listed context (Section 7: call id and
 * context id are handed to the cache engine). Advances the logical clock once per batch. For
 * each context: reactivates its ordinary messages (Section 5.2), hashes the concatenation of its
 * messages' tokens into chained block keys, walks the chain through the block table until the
 * first miss, stamps and locks the hits, and makes the new token layout the context's
 * materialised mapping. The same result as if contexts were processed one by one.
 *
 * phase KVT_MAP_ADMIT — Algorithm 1's admission test ("admit iff Delta <= 0") per 16-token block,
 * in (list order, chain order), for blocks [n_held, hit_len + n_admissible): a block already
 * resident (or inserted earlier in this batch) is adopted; otherwise it takes the lowest free
 * HBM slot; if none is free the context stops there. Eviction is the caller's job
 * (kvt_select_victims + kvt_offload) before ADMIT. May be called again to continue.
 *
 * Errors: KVT_E_NOCTX; KVT_E_INVAL duplicate context in the list, n_ctx = 0; KVT_E_STATE LOOKUP
 * on an in-flight context or ADMIT on one that is not; KVT_E_NOSPACE batch larger than
 * max_batch_blocks or key arena full. Synchronises the stream. `out` has n_ctx elements. */
int32_t kvt_map_blocks(kvt_engine *e, const uint32_t *ctx_ids, uint32_t n_ctx, uint32_t phase,
                       kvt_call_info *out, void *stream);

/* Block map of a context's materialised token sequence: key, tier (KVT_TIER_* / KVT_TIER_NONE)
 * and slot (0xFFFFFFFF if not resident) of each block as of now. Host output arrays of capacity
 * `cap`; *n receives the block count (KVT_E_BUFSZ if cap is too small). Synchronises. */
int32_t kvt_get_block_map(kvt_engine *e, uint32_t ctx, uint64_t *keys, uint8_t *tier,
                          uint32_t *slot, uint32_t cap, uint32_t *n, void *stream);

/* ---- stage 3: KV-level lifecycle state (Section 6.1, KV shared between contexts) ------------- */
/* Brings the KV-level state of every resident block up to date: the highest-priority state over all (context,
 * message version) mappings of its key; a block nobody maps is dead. The engine keeps, per block, the number of
 * mappings of each priority and updates these counts by events (Section 6.1: the aggregate is updated whenever a
 * mapped version changes state): this call applies what has happened since the last one (contexts whose messages,
 * mapped prefix or token layout changed; contexts that ended; blocks that entered the table) and touches only the
 * blocks of those contexts. Calls that need the states (selection, offload, ...) do the same on their own.
 * With KVT_POLICY_ORPHANS_DEAD the states are recomputed in full. Asynchronous on `stream`. */
int32_t kvt_classify(kvt_engine *e, void *stream);

/* Copies the ranks of one tier to a host array (KVT_STATE_FREE for empty slots); classifies
 * first if anything changed since the last classification. cap >= slots of the tier. Synchronises. */
int32_t kvt_get_states(kvt_engine *e, uint32_t tier, uint8_t *state, uint32_t cap, void *stream);

/* ---- stage 4: victim selection (Algorithm 1 order; Section 6.2 recency) ----------------------- */
/* Returns the first min(n_req, #candidates) slots of `tier` in eviction order, with their ranks.
 * Candidates: resident, not in flight, rank below Pinned (Pinned included, last, with
 * KVT_SEL_INCLUDE_PINNED). Order: rank ascending (dead, idle, active, pinned); within dead, active and
 * pinned oldest stamp first; within idle newest stamp first (MRU) or
 * oldest first if suspended_order = KVT_ORDER_LRU; then chain depth descending; then slot
 * ascending. With inclusive tiers the host tier's clean copies (KVT_STATE_COPY) come before everything
 * else, oldest first. states_out[i] is the rank, with KVT_STATE_HAS_COPY or-ed in for an HBM victim that
 * still has a clean host copy (offloading it moves no bytes and needs no host slot), or KVT_STATE_COPY.
 * With KVT_POLICY_NO_LIFECYCLE every candidate counts as rank 1. Classifies first if needed. Host output
 * arrays (states_out may be NULL). If both are pinned host memory (or device / managed memory) and
 * cap >= min(n_req, slots of the tier), the last kernel writes the list straight into them; otherwise it is staged
 * in the engine's pinned area and copied by the CPU, which for a long list costs more than the selection itself
 * (0.4 ms for 786 K victims). After an error the arrays' contents are unspecified.
 * KVT_E_BUFSZ if cap < min(n_req, #candidates). The order is computed on a packed
 * key of 2 (+1 on a host tier with clean copies) + bits(clock) + bits(largest depth) bits; KVT_E_INVAL if that exceeds
 * 63 bits (kvt_debug_load_resident refuses stamps and depths that would get there; the clock itself is 32 bits and
 * calls that would advance it past 2^32 - 1 fail with KVT_E_NOSPACE). Synchronises. */
int32_t kvt_select_victims(kvt_engine *e, uint32_t tier, uint32_t n_req, uint32_t flags, uint32_t *slots_out,
                           uint8_t *states_out, uint32_t cap, uint32_t *n_out, void *stream);

/* ---- stage 5: tier movement (Section 7; Algorithm 1 "release") -------------------------------- */
/* Processes HBM slots in the given order: a dead block is dropped (key erased, slot freed, no
 * copy; its clean host copy, if any, is freed too); a live block that has a clean host copy is handed
 * over to it (metadata only); the i-th other live block moves to the i-th lowest host slot that was
 * free when the call began, payload byte for byte, metadata carried. Stops with KVT_E_NOSPACE at the
 * first block that finds no host slot; *n_done = victims processed, *n_dropped = dead ones among them. A listed slot that is empty, out of range,
 * repeated (KVT_E_INVAL / KVT_E_RANGE) or in flight (KVT_E_STATE) rejects the whole call.
 * Host id array. Synchronises. */
int32_t kvt_offload(kvt_engine *e, const uint32_t *hbm_slots, uint32_t n, uint32_t *n_done,
                    uint32_t *n_dropped, void *stream);

/* Mirror image: the i-th listed host slot moves to the i-th lowest free HBM slot (in-flight
 * blocks allowed: a call reloads its own host hits). With inclusive tiers the host slot stays occupied
 * as the block's clean copy. A listed slot that only holds such a copy is rejected (KVT_E_INVAL).
 * KVT_E_NOSPACE + *n_done when HBM is full. Synchronises. */
int32_t kvt_reload(kvt_engine *e, const uint32_t *host_slots, uint32_t n, uint32_t *n_done,
                   void *stream);

/* Movement between neighbouring levels of the hierarchy (Section 7: HBM, host memory, remote memory) and straight
 * up from the remote tier into HBM: (HBM, host) = kvt_offload, (host, HBM) = kvt_reload, (host, remote) moves down
 * like an offload (dead blocks dropped, live ones to the remote slots that are free when the call begins, lowest
 * first; blocks in flight and clean copies are rejected), (remote, host) and (remote, HBM) move up like a reload
 * (i-th listed block to the i-th lowest free slot; blocks in flight allowed; the remote slot is freed, also with
 * inclusive tiers). Any other pair: KVT_E_INVAL. KVT_E_NOSPACE + counts when the destination fills up.
 * Host id array. Synchronises. */
int32_t kvt_move(kvt_engine *e, uint32_t src_tier, uint32_t dst_tier, const uint32_t *slots, uint32_t n,
                 uint32_t *n_done, uint32_t *n_dropped, void *stream);

/* Offload and reload in one call, for the common step "push other blocks out and bring my prefix back". Both
 * lists are validated against the state the call finds (same codes as the single calls; nothing changes on an
 * error). After that the result is by definition that of kvt_offload(hbm_slots_out) followed by
 * kvt_reload(host_slots_in): the victims are dropped / handed over / moved to the host slots that are free when the
 * call begins; the listed host blocks then take the lowest free HBM slots, those the victims just left included,
 * so the call also works on a full pool. What the single call adds: ONE mover launch carries both payload streams,
 * so they cross the host link in both directions at the same time (the link is full duplex); where a reload lands
 * in a slot a victim leaves, the same warp copies the victim's tile out before it writes the new tile in.
 * KVT_E_NOSPACE if either direction ran out of destination slots; the three counts tell how far each got.
 * Synchronises. */
int32_t kvt_exchange(kvt_engine *e, const uint32_t *hbm_slots_out, uint32_t n_out, const uint32_t *host_slots_in,
                     uint32_t n_in, uint32_t *n_out_done, uint32_t *n_dropped, uint32_t *n_in_done, void *stream);

/* Drops blocks without copying (frees host space for offloads). Same validation as kvt_offload.
 * Releasing an HBM block frees its clean host copy too; releasing a clean copy leaves its block alone. */
int32_t kvt_release(kvt_engine *e, uint32_t tier, const uint32_t *slots, uint32_t n, void *stream);

/* Hole-filling compaction inside a tier: with n_occ occupied slots, the i-th occupied slot
 * >= n_occ moves to the i-th free slot < n_occ (both ascending), so that afterwards exactly slots
 * [0, n_occ) are occupied. Metadata (including in-flight counts) is carried; callers must refresh
 * block maps. Synchronises. */
int32_t kvt_compact(kvt_engine *e, uint32_t tier, uint32_t *n_moved, void *stream);

/* Raw paged-KV mover: copies the payload of n blocks src_tier[src[i]] -> dst_tier[dst[i]]. No
 * metadata is read or changed. Id arrays are host pointers unless KVT_IDS_ON_DEVICE. Destinations
 * must be distinct and disjoint from sources within a tier (not checked); ids out of range set
 * the device error word and are skipped. n <= max_batch_blocks. Asynchronous. */
int32_t kvt_copy_blocks(kvt_engine *e, uint32_t src_tier, const uint32_t *src, uint32_t dst_tier,
                        const uint32_t *dst, uint32_t n, uint32_t flags, void *stream);

/* ---- stand-alone hasher ----------------------------------------------------------------------- */
/* Chained block keys of one token sequence, without an engine: d_keys[b], b < n_tokens/16.
 * d_tokens must be 16-byte aligned. d_scratch: device scratch of at least
 * kvt_hash_scratch_bytes(n_tokens) bytes, 8-byte aligned. Asynchronous. */
uint64_t kvt_hash_scratch_bytes(uint64_t n_tokens);
int32_t kvt_hash_tokens(const uint32_t *d_tokens, uint64_t n_tokens, uint64_t hash_seed,
                        uint64_t *d_keys, void *d_scratch, uint64_t scratch_bytes, void *stream);

/* Hasher variant for callers that cannot allocate. The paper has no counterpart for this call; it
 * exists for integrations that are handed a fixed memory budget and may not call cudaMalloc (or any
 * allocating library routine) at all: a plug-in living inside a serving engine whose allocator owns
 * every byte of the device, or a request loop in which an allocation would stall the whole device.
 * Same result as kvt_hash_tokens, but the per-chunk scratch is a fixed array inside the library
 * instead of a caller buffer, so the call allocates nothing, on the host or on the device.
 *   - d_tokens (16-byte aligned) and d_keys are device pointers supplied by the caller, as before.
 *   - Limit: n_tokens <= KVT_HASH_NOALLOC_MAX_TOKENS; larger inputs are rejected with KVT_E_NOSPACE
 *     and nothing is launched. The scratch array takes 16 KiB of device memory on every GPU that
 *     loads the library, until the process exits.
 *   - Every call asks the runtime for the array's address on the current device (no allocation). The
 *     first call on a device is the one that makes the runtime set the library up there: make that
 *     first call outside any stream capture.
 *   - All calls share the one array. Nothing in it has to start at zero (each call overwrites what it
 *     later reads), but two calls whose kernels overlap on the GPU (different streams, or different
 *     host threads) race on it: keep calls on one device ordered.
 * Asynchronous on `stream`. */
#define KVT_HASH_NOALLOC_MAX_TOKENS (1ull << 22)
int32_t kvt_hash_tokens_noalloc(const uint32_t *d_tokens, uint64_t n_tokens, uint64_t hash_seed,
                                uint64_t *d_keys, void *stream);

/* ---- introspection ------------------------------------------------------------------------------ */
typedef struct kvt_stats {
  uint64_t clock;            /* logical clock */
  uint64_t n_contexts;       /* live contexts */
  uint64_t occ_hbm, occ_host;/* occupied slots per tier */
  uint64_t blocks_hashed;    /* blocks hashed by LOOKUP */
  uint64_t hits_hbm, hits_host, misses; /* per LOOKUP block: prefix hit by tier / not in the prefix */
  uint64_t inserted;         /* blocks inserted by ADMIT */
  uint64_t adopted;          /* blocks adopted by ADMIT */
  uint64_t dropped;          /* dead blocks reclaimed without copy (offload) + released */
  uint64_t offloaded, reloaded, compacted; /* blocks moved */
  uint64_t bytes_d2h, bytes_h2d, bytes_d2d;/* payload bytes moved by offload / reload / compact */
  uint64_t table_rebuilds;
  uint64_t tombstones;
  uint64_t kernel_launches;  /* kernels of this library launched so far */
  uint64_t mover_launches;   /* with profiling on: mover kernels timed, their device time and payload bytes */
  uint64_t mover_ns;
  uint64_t mover_bytes;
  uint64_t lookup_ns;        /* with profiling on: device time of the hash + lookup + lock kernels of LOOKUP calls */
  uint64_t lookup_blocks;    /* and the blocks they processed */
  uint64_t select_ns;        /* with profiling on: device time of the selection kernels (count, compaction, sort, emit) */
  uint64_t select_slots;     /* and the tier slots they scanned */
  uint64_t offloaded_clean;  /* of `offloaded`, blocks handed to an existing clean host copy (no bytes moved) */
  uint64_t blocks_rehashed;  /* of `blocks_hashed`, blocks whose digest was actually recomputed (the rest kept their keys) */
  uint64_t occ_remote;       /* occupied slots of the remote tier */
  uint64_t hits_remote;      /* reusable-prefix blocks found in the remote tier */
  uint64_t demoted;          /* blocks moved host -> remote */
  uint64_t promoted;         /* blocks moved remote -> host or remote -> HBM */
  uint64_t classify_ns;      /* with profiling on: device time of the classification kernels */
  uint64_t classify_items;   /* and the (context, block) mappings they visited */
} kvt_stats;
int32_t kvt_get_stats(kvt_engine *e, kvt_stats *out);

/* Profiling switch (default off). When on, offload / reload / compact bracket their mover kernel with
 * CUDA events on the call's stream and accumulate its device time in kvt_stats.mover_ns. */
int32_t kvt_set_profiling(kvt_engine *e, uint32_t on);

/* Tuning hook: which mover kernel offload / reload / compact / copy_blocks launch. 0 = automatic (variant 2
 * whenever it applies, default), 1 = one CTA per (block, chunk), 2 = one warp per 4 KiB tile (needs chunk_bytes % 4096 == 0,
 * otherwise variant 1 is used), 3 = TMA bulk copies through a shared-memory ring (chunks of at most 16 KiB or a
 * multiple of 16 KiB), 4 = copy engines through the staging ring for every block size (needs kvt_config.stage_buf;
 * only offload / reload / move between device memory and a pool in host memory). With 1-3 the staging ring is not
 * used. Results are identical. */
int32_t kvt_debug_set_mover_variant(kvt_engine *e, uint32_t variant);

/* Upper bound on the thread blocks a mover kernel launches (offload / reload / exchange / move / compact /
 * copy_blocks); 0 = automatic (default): 8 blocks of 256 threads per SM for moves inside device memory; for a move
 * to or from a pool that lies in host memory 4 blocks of 1024 threads (8 for kvt_exchange, which drives both
 * directions). A move that crosses the host link is bound by the link, 128 warps keep it full, and packing them
 * into a few large blocks leaves all other SMs to kernels running on other streams at the same time. */
int32_t kvt_set_mover_ctas(kvt_engine *e, uint32_t max_ctas);

/* Tuning hook: how kvt_map_blocks(LOOKUP) hashes and probes. 0 / 1 = two kernels (digest; chunk carry + finish +
 * probe; default), 2 = one single-pass kernel in which chunks hand their chain values forward through device
 * memory (bounded waits; a wait that runs out makes the call return KVT_E_DEVICE), 3 / 4 = the default kernels with
 * one / four keys per thread in the probe instead of two. Results are identical; on B200 the single pass measured
 * slower (its CTAs live too long to keep enough token bytes in flight) and the other probe widths within 3 % of the
 * default. */
int32_t kvt_debug_set_lookup_variant(kvt_engine *e, uint32_t variant);

/* L2 residency of the metadata (default on where the device supports it): the kernels that probe the block table and
 * the per-entry arrays are launched with an access-policy window over them, so those lines sit in the persisting part
 * of L2 (up to the device's maximum, 79 MiB on B200; the process-wide limit cudaLimitPersistingL2CacheSize is raised to
 * what the engine needs, never lowered) while KV payload and token streams, which are read and written with
 * streaming accesses, pass through the rest. 0 switches it off and gives the persisting lines back. */
int32_t kvt_set_l2_residency(kvt_engine *e, uint32_t on);

/* Test hook for the ordering of a call's kernels: the small kernels that carry a call's control records between the
 * pinned staging area and the device start their copy delay_ns later (at most 1,000,000). Results must not depend on
 * it; a kernel of the same call that read a record before it is entitled to would see the previous call's. */
int32_t kvt_debug_set_copy_delay(kvt_engine *e, uint32_t delay_ns);

/* Test / measurement hook for the classification: 0 = event-driven (default), 1 = every kvt_classify recomputes all
 * counts from zero over all contexts, 2 = event-driven, and every update is followed by a full recomputation that must
 * give the same counts (KVT_E_DEVICE if not). */
int32_t kvt_debug_set_classify_mode(kvt_engine *e, uint32_t mode);

/* Test hook for the bounded wait of the single-pass lookup (variant 2): the number of polls a chunk spends on its
 * predecessors' publications before it gives up (default 2^18). With 0 every chunk that needs a predecessor gives
 * up at once: the kernel still returns normally, the call reports KVT_E_DEVICE and the engine is unchanged. */
int32_t kvt_debug_set_wait_limit(kvt_engine *e, uint32_t polls);

/* Text of the last error of this engine (always NUL-terminated). */
int32_t kvt_last_error(kvt_engine *e, char *buf, uint32_t cap);

/* Copies per-slot metadata of a tier to host arrays (any may be NULL): key (0 = free), stamp,
 * depth, in-flight count, and link = the slot of the other tier that holds this block's clean copy /
 * the block this copy belongs to (0xFFFFFFFF: none). cap >= slots of the tier. Synchronises. */
int32_t kvt_get_entries(kvt_engine *e, uint32_t tier, uint64_t *keys, uint32_t *stamp,
                        uint32_t *depth, uint32_t *inflight, uint32_t *link, uint32_t cap, void *stream);

/* Test / benchmark hook: makes n blocks resident in `tier` at the given slots without running
 * calls. state[i] acts as a permanent anonymous mapping of that rank (classification never reports
 * less for the block until it is dropped). Keys must be >= 2, distinct and not resident; slots
 * free and distinct, and 3 + bits(max stamp) + bits(max depth) <= 63 (violations: KVT_E_INVAL, state unchanged).
 * Advances the logical clock to at least max(stamp). Host arrays. Synchronises. */
int32_t kvt_debug_load_resident(kvt_engine *e, const uint64_t *keys, const uint8_t *state,
                                const uint32_t *stamp, const uint32_t *depth,
                                const uint32_t *slot, uint32_t tier, uint32_t n, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* KVT_H_ */
