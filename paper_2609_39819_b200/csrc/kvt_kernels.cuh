// kvt_kernels.cuh — sm_100a kernels of the KV-cache hot path: block hasher, open-addressing block
// table, lifecycle classifier, victim selection (ordered compaction + LSD radix sort) and paged KV
// mover. Host-side launch logic lives in kvt_engine.cu.
//
// Conventions: every probe loop is capped at the table capacity and reports through the status
// word (never traps, never spins on another thread's progress); there are no inter-CTA waits, so
// every multi-pass algorithm is a sequence of kernels. No tensor cores: nothing here is a dense
// contraction.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace kvt {

typedef uint8_t u8;
typedef uint32_t u32;
typedef uint64_t u64;

constexpr u64 KEY_EMPTY = 0, KEY_TOMB = 1;
constexpr u32 ENT_NONE = 0xFFFFFFFFu;
constexpr u32 CLAIM_BIT = 0x80000000u;
constexpr u32 CHUNK = 256;        // blocks hashed by one CTA
constexpr u32 SCAN_TILE = 1024;   // items per CTA in the ordered-compaction kernels

// bits of the device error word
enum : u32 { DERR_PROBE = 1, DERR_RANGE = 2, DERR_INVAL = 4, DERR_STATE = 8, DERR_CORRUPT = 16, DERR_WAIT = 32 };

// words of the device status block
enum : int {
  ST_ERR = 0, ST_TOTAL, ST_CUT, ST_NLIVE, ST_NDROP, ST_NEW, ST_INSERTED, ST_ADOPTED, ST_TOMBS,
  ST_RANK0, ST_RANK1, ST_RANK2, ST_RANK3, ST_M, ST_NMOVED, ST_FREE, ST_AUX, ST_SHADOW, ST_NCLEAN, ST_NSHDROP,
  ST_B_CUT, ST_B_NLIVE, ST_B_NDROP, ST_B_NCLEAN, ST_B_NSHDROP, ST_B_TOTAL, ST_B_FREE,   // second list of an exchange
  ST_QA, ST_QB,                                                                          // work queues of its mover
  ST_CHK,                                                                                // cross-check of the mapping counts
  ST_WORDS = 32
};

struct __align__(16) TSlot { u64 key; u32 ent; u32 pad; };

// ---- hash constants (compile-time; only H0 depends on the seed) -------------------------------------
__host__ __device__ constexpr u64 mix64(u64 z) {
  z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull;
  z ^= z >> 27; z *= 0x94D049BB133111EBull;
  z ^= z >> 31;
  return z;
}
constexpr u64 GOLD = 0x9E3779B97F4A7C15ull;
constexpr u64 HASH_P = mix64(GOLD * 17ull) | 1ull;
__host__ __device__ constexpr u64 lane_mult(u32 t) { return mix64(GOLD * (u64)(t + 1)) | 1ull; }
__host__ __device__ constexpr u64 hash_h0(u64 seed) { return mix64(seed ^ (GOLD * 18ull)); }

__host__ __device__ __forceinline__ u64 pow_u64(u64 b, u32 e) {
  u64 r = 1;
  while (e) { if (e & 1) r *= b; b *= b; e >>= 1; }
  return r;
}
__host__ __device__ __forceinline__ u64 pow_p(u32 e) { return pow_u64(HASH_P, e); }

// P^0 .. P^CHUNK, constant-initialised at compile time (2 KiB, L1-resident).
struct PowTable {
  u64 v[CHUNK + 1];
  constexpr PowTable() : v() { u64 p = 1; for (u32 i = 0; i <= CHUNK; ++i) { v[i] = p; p *= HASH_P; } }
};
__device__ const PowTable g_pow_p = PowTable();
// A^0 .. A^64 with A = P^CHUNK: the weights of the chunk aggregates of sequences of up to 64 chunks (16 Ki blocks);
// longer ones fall back to square-and-multiply.
struct ChunkPowTable {
  u64 v[65];
  constexpr ChunkPowTable() : v() {
    u64 a = 1;
    for (u32 i = 0; i < CHUNK; ++i) a *= HASH_P;
    u64 p = 1;
    for (u32 i = 0; i <= 64; ++i) { v[i] = p; p *= a; }
  }
};
__device__ const ChunkPowTable g_pow_a = ChunkPowTable();
__device__ __forceinline__ u64 pow_a(u32 e) { return e <= 64 ? g_pow_a.v[e] : pow_u64(g_pow_p.v[CHUNK], e); }

// ---- device views -------------------------------------------------------------------------------------
struct Table { TSlot *slots; u32 mask; u32 shift; };   // capacity = mask + 1, home = key >> shift

struct Entries {            // per resident-block metadata, entry id = slot (HBM), n_hbm + slot (host) or n_hbm + n_host + slot (remote)
  u64 *key;                 // 0 = free
  u32 *stamp, *depth, *infl, *tslot, *mark;
  u64 *cnt;                 // mappings per rank: three 21-bit fields (Suspended, Active, Pinned), see entry_rank()
  u32 *link;                // inclusive tiering: an HBM block and its clean host copy point at each other (else ENT_NONE)
  u8 *floor;
  u32 n_hbm, n_host, n_total;
};

// KV-level state of a resident block (Section 6.1): the highest-priority state over all (context, message version)
// mappings of its key, dead when there is none. cnt[e] counts the mappings per rank, so the state is the highest
// rank with a non-zero count (or the floor installed by the debug loader, whichever is higher).
constexpr u32 CNT_BITS = 21;
constexpr u64 CNT_MASK = (1ull << CNT_BITS) - 1;
__host__ __device__ __forceinline__ u64 cnt_unit(u32 rank) { return rank ? 1ull << (CNT_BITS * (rank - 1)) : 0ull; }
__device__ __forceinline__ u32 rank_of(u64 cnt, u32 floor) {
  const u32 r = (cnt >> (2 * CNT_BITS)) ? 3u : ((cnt >> CNT_BITS) & CNT_MASK) ? 2u : (cnt & CNT_MASK) ? 1u : 0u;
  return max(r, floor);
}
__device__ __forceinline__ u32 entry_rank(const Entries &en, u32 e) { return rank_of(en.cnt[e], en.floor[e]); }

// A host entry that only holds a clean copy of a block whose home is in HBM.
__device__ __forceinline__ bool is_shadow(const Entries &en, u32 e) { return e >= en.n_hbm && en.link[e] != ENT_NONE; }

__device__ __forceinline__ void set_err(u32 *status, u32 bits) { atomicOr(&status[ST_ERR], bits); }

// Index and invariant checks of the checked build (-DKVT_DEBUG): a violation sets the error word and skips the
// access (never a trap, never a wild store); the call then reports KVT_E_DEVICE. They compile to nothing otherwise.
#ifdef KVT_DEBUG
#define KVT_CHECK(cond, status, action) do { if (!(cond)) { set_err((status), DERR_CORRUPT); action; } } while (0)
#else
#define KVT_CHECK(cond, status, action) do { } while (0)
#endif

// Home slot of a key: the even slot of the pair its top bits select. Probe sequences start at an aligned pair, so
// every two-slot step of a read-only probe reads one 32-byte sector.
__device__ __forceinline__ u32 tab_home(const Table &t, u64 key) { return (u32)(key >> t.shift) & ~1u; }

// Finds key; returns its table slot index or ENT_NONE. Stops at the first EMPTY slot.
__device__ __forceinline__ u32 tab_find(const Table &t, u64 key, u32 *status) {
  u32 i = tab_home(t, key);
  for (u32 n = 0; n <= t.mask; ++n, i = (i + 1) & t.mask) {
    u64 k = t.slots[i].key;
    if (k == key) return i;
    if (k == KEY_EMPTY) return ENT_NONE;
  }
  set_err(status, DERR_PROBE);
  return ENT_NONE;
}

// Read-only probe for kernels that run while nobody writes the table: returns the entry id stored for key, or
// ENT_NONE. Each step fetches two consecutive slots with two independent 16-byte loads (key and entry id come
// together), so a probe sequence of length p costs ceil(p / 2) dependent memory round trips and no extra one for
// the entry id.
__device__ __forceinline__ u32 tab_lookup_ent(const Table &t, u64 key, u32 *status) {
  u32 i = tab_home(t, key);
  for (u32 n = 0; n <= t.mask; n += 2) {
    const uint4 a = __ldg(reinterpret_cast<const uint4 *>(t.slots + i));
    const uint4 b = __ldg(reinterpret_cast<const uint4 *>(t.slots + ((i + 1) & t.mask)));
    const u64 ka = (u64)a.x | ((u64)a.y << 32), kb = (u64)b.x | ((u64)b.y << 32);
    if (ka == key) return a.z;
    if (ka == KEY_EMPTY) return ENT_NONE;
    if (kb == key) return b.z;
    if (kb == KEY_EMPTY) return ENT_NONE;
    i = (i + 2) & t.mask;
  }
  set_err(status, DERR_PROBE);
  return ENT_NONE;
}

// Finds key or claims the first EMPTY slot of its probe sequence for it (tombstones are skipped,
// never reused, so two threads inserting the same key always meet in the same slot).
__device__ __forceinline__ u32 tab_find_or_claim(const Table &t, u64 key, u32 *status) {
  u32 i = tab_home(t, key);
  for (u32 n = 0; n <= t.mask;) {
    u64 k = *(volatile u64 *)&t.slots[i].key;
    if (k == key) return i;
    if (k == KEY_EMPTY) {
      u64 old = atomicCAS((unsigned long long *)&t.slots[i].key, (unsigned long long)KEY_EMPTY,
                          (unsigned long long)key);
      if (old == KEY_EMPTY || old == key) return i;
      // somebody else took the slot for another key: move on
    }
    ++n; i = (i + 1) & t.mask;
  }
  set_err(status, DERR_PROBE);
  return ENT_NONE;
}

// ======================================================================================================
// K1: block hasher. Two kernels, no inter-CTA waits:
//   digest : per 256-block chunk, 4 lanes per block read 16 B each, weighted sums, mix, then a CTA-wide
//            scan of the affine chain with zero carry-in -> partial chain values + chunk aggregate
//   finish : every chunk's CTA folds the aggregates of the chunks before it into the chain value entering its
//            chunk (carry), then h = P^(i+1) * carry + partial, key = mix64(h); fused with the table probe
// Incremental: a sequence whose leading blocks are unchanged since its previous key list only digests from the
// last chunk boundary before the first changed block (the chain restarts from the carry kept for that chunk).
// ======================================================================================================
// One sequence of a batch. Blocks [0, first) keep the keys of the previous key list (first is a multiple of
// CHUNK): only chunks from first / CHUNK on are digested, restarting the chain from the carry stored for that
// chunk. The per-chunk carries of a sequence are kept next to its keys for exactly this purpose.
struct HashCtx {
  u64 tok_off;        // token buffer (u32 index into HashArgs.tokens)
  u64 key_off;        // key list (u64 index into HashArgs.keys)
  u64 carry_off;      // per-chunk carries (u64 index into HashArgs.carry_base)
  u64 old_key_off;    // previous key list and carries, read when first > 0
  u64 old_carry_off;
  u32 n_blocks;
  u32 first;
  u32 chunk_base;     // first chunk of this sequence in the all-blocks grid (finish / lock kernels)
  u32 dchunk_base;    // first chunk in the digest grid (chunks >= first / CHUNK only)
  u32 blk_base;       // first block of this sequence in the batch-wide result arrays
  u32 pad;
};

struct HashArgs {
  const u32 *tokens; u64 *keys; u64 *carry_base; const HashCtx *ctx; HashCtx single; u32 n_ctx;
  u64 *agg; u64 h0;
  const u32 *chunk_ctx, *dchunk_ctx;   // batch only: sequence index of every chunk of the all-blocks / digest grid
  u32 carries_ready;   // the chunk carries were written by k_hash_carry (long sequences): the finish kernel reads them
};

// Sequence that owns chunk `chunk` of the all-blocks grid (dgrid = false) or of the digest grid (dgrid = true):
// looked up in the chunk -> sequence map the host uploads with the descriptors (two dependent loads, no search).
__device__ __forceinline__ const HashCtx &hash_ctx_of_chunk(const HashArgs &a, u32 chunk, u32 *ctx_idx, bool dgrid = false) {
  if (!a.ctx) { *ctx_idx = 0; return a.single; }
  const u32 i = dgrid ? a.dchunk_ctx[chunk] : a.chunk_ctx[chunk];
  *ctx_idx = i;
  return a.ctx[i];
}

// Lane multipliers K[0..15] as a constant-initialised table (read once per thread, L1-resident).
struct LaneTable {
  u64 v[16];
  constexpr LaneTable() : v() { for (u32 t = 0; t < 16; ++t) v[t] = lane_mult(t); }
};
__device__ const LaneTable g_lane_mult = LaneTable();

// Block digests of one 256-block chunk from the quad layout (lane q of a quad holds tokens 4q..4q+3 of the blocks
// it*64 + tid/4, it = 0..3): weighted sums, quad reduction, mix; sd[blk] = d_blk (0 beyond nb).
__device__ __forceinline__ void digest_quads(const uint4 (&v)[4], u32 q, u64 k0, u64 k1, u64 k2, u64 k3, u64 ksum,
                                             u32 tid, u32 nb, u64 *sd) {
  // per iteration: low words of the multipliers through widening multiply-adds into one 64-bit accumulator, high
  // words through 32-bit multiply-adds into one 32-bit accumulator (tok * K mod 2^64 = tok*Klo + ((tok*Khi) << 32))
  const u32 k0l = (u32)k0, k1l = (u32)k1, k2l = (u32)k2, k3l = (u32)k3;
  const u32 k0h = (u32)(k0 >> 32), k1h = (u32)(k1 >> 32), k2h = (u32)(k2 >> 32), k3h = (u32)(k3 >> 32);
  u64 part[4];
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    u64 lo = ksum;
    lo += (u64)v[it].x * k0l; lo += (u64)v[it].y * k1l; lo += (u64)v[it].z * k2l; lo += (u64)v[it].w * k3l;
    u32 hi = v[it].x * k0h + v[it].y * k1h + v[it].z * k2h + v[it].w * k3h;
    part[it] = lo + ((u64)hi << 32);
  }
  // quad reduction that leaves lane q with the block of iteration q: two exchange steps, each lane passing on the
  // halves it does not keep (3 64-bit shuffles instead of 8)
  {
    const bool up2 = q & 2, up1 = q & 1;
    u64 keep0 = up2 ? part[2] : part[0], keep1 = up2 ? part[3] : part[1];
    u64 send0 = up2 ? part[0] : part[2], send1 = up2 ? part[1] : part[3];
    keep0 += __shfl_xor_sync(0xFFFFFFFFu, send0, 2);
    keep1 += __shfl_xor_sync(0xFFFFFFFFu, send1, 2);
    u64 keep = up1 ? keep1 : keep0, send = up1 ? keep0 : keep1;
    keep += __shfl_xor_sync(0xFFFFFFFFu, send, 1);
    u32 blk = (q * CHUNK + tid) >> 2;
    sd[blk] = blk < nb ? mix64(keep) : 0;
  }
}

// ---- untiled bulk copies (cp.async.bulk) and the mbarriers they complete on; every wait is bounded -----------
constexpr u32 TMA_WAIT_LIMIT = 1u << 20;

__device__ __forceinline__ u32 smem_u32(const void *p) { return (u32)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(u64 *bar, u32 count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(u64 *bar, u32 bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Polls the barrier's phase; gives up after TMA_WAIT_LIMIT polls (returns false).
__device__ __forceinline__ bool mbar_wait(u64 *bar, u32 parity) {
  u32 done = 0;
  for (u32 n = 0; n < TMA_WAIT_LIMIT && !done; ++n) {
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  }
  return done != 0;
}
__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gsrc, u32 bytes, u64 *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bulk_store(void *gdst, const void *smem_src, u32 bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

// Dependent launches inside one call: a kernel releases the next launch of its stream at its start (the next
// kernel's CTAs then fill the SM slots this kernel's tail leaves free), and the next kernel waits, before it touches
// anything this one writes, until this grid has finished and its writes are visible. Both are no-ops for a launch
// without the attribute. In a chain A -> B -> C of such launches C may start while B still waits for A, so a kernel
// of a chain reads nothing that any earlier kernel of the chain writes before its own wait, and every CTA waits
// (then "B has finished" implies "A has finished").
__device__ __forceinline__ void dep_release() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Chain values of a chunk with zero carry-in from its block digests sd[] (an inclusive scan of
// c_t = sum_{i<=t} P^(t-i) d_i over the CTA), stored where the keys will be; the last one is the chunk's aggregate.
__device__ __forceinline__ void chunk_scan_store(const HashArgs &a, const HashCtx &c, u32 b0, u32 nb, u32 dchunk, const u64 *sd,
                                                 u64 *wagg) {
  const u32 tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  u64 cval = sd[tid];
  u64 pp = HASH_P;
#pragma unroll
  for (u32 o = 1; o < 32; o <<= 1) {
    u64 up = __shfl_up_sync(0xFFFFFFFFu, cval, o);
    if (lane >= o) cval += pp * up;
    pp *= pp;
  }
  if (lane == 31) wagg[warp] = cval;
  __syncthreads();
  u64 carry = 0;  // chain value at the end of the previous warp, with zero chunk carry-in
  const u64 p32 = pp;  // after 5 squarings pp = P^32
  for (u32 w = 0; w < warp; ++w) carry = p32 * carry + wagg[w];
  cval += g_pow_p.v[lane + 1] * carry;
  if (tid < nb) a.keys[c.key_off + b0 + tid] = cval;
  if (tid == nb - 1) a.agg[dchunk] = cval;
}

// Small control records between the pinned staging area and device memory (either direction; both are in the
// device's address space): the descriptors of a call going up, status and result words coming back. A kernel
// reaches a few tens of KB over the host link in about a third of the time a copy-engine transfer of that size
// takes to start and finish, and it can be a dependent launch on both sides.
// delay_ns (a test hook, at most a millisecond): the copy starts that much later, so that a kernel launched behind
// it which looks at the records before it is entitled to sees the previous call's.
__device__ __forceinline__ void copy_delay(u32 delay_ns) {
  if (!delay_ns) return;
  u64 t0, t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
  do { asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); } while (t - t0 < delay_ns);
}
__global__ void __launch_bounds__(256) k_copy_words(const uint4 *src, uint4 *dst, u32 n16, u32 delay_ns) {
  dep_release();
  dep_wait();
  copy_delay(delay_ns);
  for (u32 i = blockIdx.x * 256 + threadIdx.x; i < n16; i += gridDim.x * 256) dst[i] = src[i];
}

// The same for up to six stretches at once, of any alignment (16-byte, 4-byte or single-byte steps).
struct CopySegs { const void *src[6]; void *dst[6]; u32 bytes[6]; u32 n; };
__global__ void __launch_bounds__(256) k_copy_segs(CopySegs c, u32 delay_ns) {
  dep_release();
  dep_wait();
  copy_delay(delay_ns);
  const u32 t = blockIdx.x * 256 + threadIdx.x, T = gridDim.x * 256;
  for (u32 k = 0; k < c.n; ++k) {
    const uintptr_t both = (uintptr_t)c.src[k] | (uintptr_t)c.dst[k] | c.bytes[k];
    if (!(both & 15)) {
      const uint4 *s = (const uint4 *)c.src[k]; uint4 *d = (uint4 *)c.dst[k];
      for (u32 i = t; i < c.bytes[k] / 16; i += T) d[i] = s[i];
    } else if (!(both & 3)) {
      const u32 *s = (const u32 *)c.src[k]; u32 *d = (u32 *)c.dst[k];
      for (u32 i = t; i < c.bytes[k] / 4; i += T) d[i] = s[i];
    } else {
      const u8 *s = (const u8 *)c.src[k]; u8 *d = (u8 *)c.dst[k];
      for (u32 i = t; i < c.bytes[k]; i += T) d[i] = s[i];
    }
  }
}

__global__ void __launch_bounds__(CHUNK) k_hash_digest(HashArgs a) {
  __shared__ u64 sd[CHUNK];
  __shared__ u64 wagg[CHUNK / 32];
  dep_release();
  dep_wait();   // the descriptors, when the kernel that brings them up is the launch before this one
  const u32 tid = threadIdx.x;
  u32 ci;
  const HashCtx c = hash_ctx_of_chunk(a, blockIdx.x, &ci, true);
  const u32 b0 = c.first + (blockIdx.x - c.dchunk_base) * CHUNK;
  const u32 nb = min(CHUNK, c.n_blocks - b0);
  const uint4 *tok = reinterpret_cast<const uint4 *>(a.tokens + c.tok_off + (u64)b0 * 16);
  const u32 q = tid & 3;
  const u64 k0 = g_lane_mult.v[4 * q], k1 = g_lane_mult.v[4 * q + 1], k2 = g_lane_mult.v[4 * q + 2],
            k3 = g_lane_mult.v[4 * q + 3];
  const u64 ksum = k0 + k1 + k2 + k3;   // sum (tok + 1) K = sum tok K + sum K
  uint4 v[4];
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    u32 idx = it * CHUNK + tid;
    v[it] = (idx >> 2) < nb ? __ldcs(tok + idx) : make_uint4(0, 0, 0, 0);   // read once: evict-first
  }
  // iteration `it` covers blocks it*64 .. it*64+63, four lanes per block; after the two exchange steps every
  // lane of a quad holds the four block sums, and lane q finishes the block of iteration q
  digest_quads(v, q, k0, k1, k2, k3, ksum, tid, nb, sd);
  __syncthreads();
  chunk_scan_store(a, c, b0, nb, blockIdx.x, sd, wagg);
}

struct LookupArgs {
  Table tab;            // slots == nullptr: hash only
  u32 *b_ent;           // per batch block: entry id or ENT_NONE
  u32 *hit_len;         // per context, pre-initialised to n_blocks
  u32 *status;
};

// Read-only probes of ILP keys at once: the first two slots of every key are fetched before any of them is looked
// at (2 * ILP independent 16-byte loads in flight per thread), later steps only for the keys still unresolved.
template <int ILP>
__device__ __forceinline__ void tab_lookup_ents(const Table &t, const u64 (&key)[ILP], const bool (&active)[ILP], u32 (&ent)[ILP],
                                                u32 *status) {
  u32 i[ILP];
  bool open[ILP];
  bool any = false;
#pragma unroll
  for (int q = 0; q < ILP; ++q) { i[q] = tab_home(t, key[q]); open[q] = active[q]; ent[q] = ENT_NONE; any = any || open[q]; }
  for (u32 n = 0; any && n <= t.mask; n += 2) {
    uint4 a[ILP], b[ILP];
#pragma unroll
    for (int q = 0; q < ILP; ++q)
      if (open[q]) {
        a[q] = __ldg(reinterpret_cast<const uint4 *>(t.slots + i[q]));
        b[q] = __ldg(reinterpret_cast<const uint4 *>(t.slots + ((i[q] + 1) & t.mask)));
      }
    any = false;
#pragma unroll
    for (int q = 0; q < ILP; ++q)
      if (open[q]) {
        const u64 ka = (u64)a[q].x | ((u64)a[q].y << 32), kb = (u64)b[q].x | ((u64)b[q].y << 32);
        if (ka == key[q]) { ent[q] = a[q].z; open[q] = false; }
        else if (ka == KEY_EMPTY) open[q] = false;
        else if (kb == key[q]) { ent[q] = b[q].z; open[q] = false; }
        else if (kb == KEY_EMPTY) open[q] = false;
        else { i[q] = (i[q] + 2) & t.mask; any = true; }
      }
  }
  if (any) set_err(status, DERR_PROBE);
}

// Chain value entering chunk j of a sequence (j counted from the first digested chunk g0 = first / CHUNK):
// A^m C0 + sum_{i<m} A^(m-1-i) agg_i with m = j - g0, A = P^CHUNK (every chunk before the last is full) and C0 the
// value entering chunk g0 (H0, or the carry kept from the previous key list). Every thread of the CTA calls it;
// the terms are spread over the threads and summed.
template <u32 T>
__device__ __forceinline__ u64 chunk_carry(const HashArgs &a, const HashCtx &c, u32 j) {
  __shared__ u64 s_part[T / 32];
  const u32 g0 = c.first / CHUNK, m = j - g0, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  u64 sum = 0;
  for (u32 i = tid; i < m; i += T) sum += pow_a(m - 1 - i) * a.agg[c.dchunk_base + i];
  if (tid == 0) sum += pow_a(m) * (g0 ? a.carry_base[c.old_carry_off + g0] : a.h0);
#pragma unroll
  for (u32 o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
  if (lane == 0) s_part[warp] = sum;
  __syncthreads();
  u64 total = 0;
#pragma unroll
  for (u32 w = 0; w < T / 32; ++w) total += s_part[w];
  return total;
}

// The chunk carries of every sequence by a scan, one CTA per sequence: used instead of the fold above when a sequence
// has more than FOLD_MAX_CHUNKS chunks to digest (the fold reads every aggregate before a chunk, which is quadratic
// in the sequence length: 64 Mi tokens are 16,384 chunks). Also copies the kept carries and writes the resume point.
constexpr u32 FOLD_MAX_CHUNKS = 128;
__global__ void __launch_bounds__(1024) k_hash_carry(HashArgs a) {
  __shared__ u64 wtot[32], wpre[32], sv[1024];
  const u32 i = blockIdx.x;
  if (i >= a.n_ctx) return;
  const u32 tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const HashCtx c = a.ctx ? a.ctx[i] : a.single;
  const u32 g0 = c.first / CHUNK;
  const u32 n_chunks = (c.n_blocks - c.first + CHUNK - 1) / CHUNK;   // chunks that were digested
  for (u32 k = tid; k < g0; k += 1024) a.carry_base[c.carry_off + k] = a.carry_base[c.old_carry_off + k];
  const u64 A = g_pow_p.v[CHUNK];
  const u64 A32 = pow_u64(A, 32);
  const u64 a_lane = pow_u64(A, lane + 1);          // A^(lane+1)
  const u64 a_tid = pow_u64(A32, warp) * a_lane;    // A^(tid+1)
  u64 carry = g0 ? a.carry_base[c.old_carry_off + g0] : a.h0;
  if (n_chunks == 0 && tid == 0) a.carry_base[c.carry_off + g0] = carry;   // nothing new: keep the resume point
  for (u32 base = 0; base < n_chunks; base += 1024) {
    const u32 j = base + tid;
    u64 x = j < n_chunks ? a.agg[c.dchunk_base + j] : 0;
    u64 pp = A;
#pragma unroll
    for (u32 o = 1; o < 32; o <<= 1) {
      u64 up = __shfl_up_sync(0xFFFFFFFFu, x, o);
      if (lane >= o) x += pp * up;
      pp *= pp;
    }
    if (lane == 31) wtot[warp] = x;
    __syncthreads();
    if (warp == 0) {   // value at the end of every earlier warp of this round, with zero carry-in
      u64 y = wtot[lane], qq = A32;
#pragma unroll
      for (u32 o = 1; o < 32; o <<= 1) {
        u64 up = __shfl_up_sync(0xFFFFFFFFu, y, o);
        if (lane >= o) y += qq * up;
        qq *= qq;
      }
      u64 e = __shfl_up_sync(0xFFFFFFFFu, y, 1);
      wpre[lane] = lane ? e : 0;
    }
    __syncthreads();
    sv[tid] = a_tid * carry + a_lane * wpre[warp] + x;   // chain value after chunk g0 + j
    __syncthreads();
    if (j < n_chunks) a.carry_base[c.carry_off + g0 + j] = tid ? sv[tid - 1] : carry;
    // value after the last chunk: the resume point of a later call if that chunk is full
    if (j == n_chunks - 1) a.carry_base[c.carry_off + g0 + n_chunks] = sv[tid];
    carry = sv[1023];
    __syncthreads();
  }
}

// One CTA of CHUNK / ILP threads per 256-block chunk; thread t finishes and probes blocks t, t + CHUNK / ILP, ...
// The CTA first works out the chain value entering its chunk from the chunk aggregates of the digest kernel (no
// separate scan kernel) and stores it next to the keys, where a later call resumes from it.
template <int ILP>
__global__ void __launch_bounds__(CHUNK / ILP) k_hash_finish_lookup(HashArgs a, LookupArgs l) {
  constexpr u32 T = CHUNK / ILP;
  const u32 tid = threadIdx.x;
  // Nothing is read before the wait, not even the descriptors: a dependent launch may start as soon as the grid
  // before it has started, and that grid may itself still be waiting for the kernel that brings the descriptors up.
  dep_release();
  dep_wait();
  u32 ci;
  const HashCtx c = hash_ctx_of_chunk(a, blockIdx.x, &ci);
  const u32 j = blockIdx.x - c.chunk_base;
  const u32 b0 = j * CHUNK;
  const u32 nb = min(CHUNK, c.n_blocks - b0);
  u64 key[ILP];
  bool act[ILP];
  const bool kept = b0 < c.first;                                   // unchanged prefix: the keys of the previous list still hold
  u64 carry = 0;
  u64 loc[ILP];   // chain values with zero carry-in (or, in the unchanged prefix, the old keys): fetched before the carry is known
#pragma unroll
  for (int q = 0; q < ILP; ++q) {
    const u32 jj = tid + q * T;
    loc[q] = jj < nb ? a.keys[(kept ? c.old_key_off : c.key_off) + b0 + jj] : 0;
  }
  if (a.carries_ready) {
    if (!kept) carry = a.carry_base[c.carry_off + j];
  } else if (kept) {
    if (tid == 0) {
      a.carry_base[c.carry_off + j] = a.carry_base[c.old_carry_off + j];
      if (b0 + CHUNK == c.n_blocks) a.carry_base[c.carry_off + j + 1] = a.carry_base[c.old_carry_off + j + 1];   // nothing new: the resume point
    }
  } else {
    carry = chunk_carry<T>(a, c, j);
    if (tid == 0) {
      a.carry_base[c.carry_off + j] = carry;
      if (b0 + nb == c.n_blocks)   // value after the last chunk: the resume point of a later call if that chunk is full
        a.carry_base[c.carry_off + j + 1] = g_pow_p.v[nb] * carry + a.agg[c.dchunk_base + (j - c.first / CHUNK)];
    }
  }
#pragma unroll
  for (int q = 0; q < ILP; ++q) {
    const u32 jj = tid + q * T;
    act[q] = jj < nb;
    key[q] = 0;
    if (act[q]) {
      if (kept) key[q] = loc[q];
      else {
        key[q] = mix64(g_pow_p.v[jj + 1] * carry + loc[q]);
        if (key[q] < 2) key[q] += 2;
      }
      a.keys[c.key_off + b0 + jj] = key[q];
    }
  }
  if (!l.tab.slots) return;
  u32 ent[ILP];
  tab_lookup_ents<ILP>(l.tab, key, act, ent, l.status);
  u32 miss = 0xFFFFFFFFu;
#pragma unroll
  for (int q = 0; q < ILP; ++q)
    if (act[q]) {
      const u32 jj = tid + q * T;
      l.b_ent[c.blk_base + b0 + jj] = ent[q];
      if (ent[q] == ENT_NONE) miss = min(miss, b0 + jj);
    }
  // first miss of the CTA -> the context's reusable prefix length: warp minima meet in shared memory, one global
  // atomic per CTA that saw a miss
  __shared__ u32 s_min;
  if (tid == 0) s_min = 0xFFFFFFFFu;
  __syncthreads();
  miss = __reduce_min_sync(0xFFFFFFFFu, miss);
  if ((tid & 31) == 0 && miss != 0xFFFFFFFFu) atomicMin(&s_min, miss);
  __syncthreads();
  if (tid == 0 && s_min != 0xFFFFFFFFu) atomicMin(&l.hit_len[ci], s_min);
}

// ------------------------------------------------------------------------------------------------------
// Single-pass form of digest + carry + finish + probe for a LOOKUP batch. A CTA takes the next chunk of the
// all-blocks grid from a ticket counter (so every chunk with a lower number is already running or done),
// digests it, publishes its aggregate, finds the chain value entering it by looking back over the
// aggregates / chain values its predecessors of the same sequence have published (32 predecessors per step,
// folded as affine maps), publishes its own chain value and finishes + probes its 256 keys. The streaming
// token reads of some chunks overlap the random table reads of others. Every wait is bounded: a CTA that
// gives up sets DERR_WAIT and carries on with a zero carry (the call then fails; no table word is written by
// this kernel).
// ------------------------------------------------------------------------------------------------------
struct ChainState {
  u32 *flags;    // per chunk of the all-blocks grid: 0 nothing, 1 aggregate published, 2 chain value published
  u64 *incl;     // chain value after the chunk
  u32 *ticket;   // next chunk to hand out (zero at launch, like the flags)
  u32 spin_limit;
};

__device__ __forceinline__ u32 ld_acquire_u32(const u32 *p) {
  u32 v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_u32(u32 *p, u32 v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

__global__ void __launch_bounds__(CHUNK) k_hash_lookup_fused(HashArgs a, LookupArgs l, ChainState cs) {
  __shared__ u64 sd[CHUNK];
  __shared__ u64 wagg[CHUNK / 32];
  __shared__ u64 s_carry;
  __shared__ u32 s_chunk, s_min;
  const u32 tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { s_chunk = atomicAdd(cs.ticket, 1u); s_min = 0xFFFFFFFFu; }
  __syncthreads();
  const u32 chunk = s_chunk;
  u32 ci;
  const HashCtx c = hash_ctx_of_chunk(a, chunk, &ci);
  const u32 j = chunk - c.chunk_base;            // chunk index inside the sequence
  const u32 b0 = j * CHUNK;
  const u32 nb = min(CHUNK, c.n_blocks - b0);
  const u32 g0 = c.first / CHUNK;
  u64 key = 0;
  if (b0 < c.first) {
    // unchanged prefix: keys and the carry entering this chunk are taken over from the previous list
    if (tid < nb) key = a.keys[c.old_key_off + b0 + tid];
    if (tid == 0) {
      a.carry_base[c.carry_off + j] = a.carry_base[c.old_carry_off + j];
      if (b0 + CHUNK == c.n_blocks) a.carry_base[c.carry_off + j + 1] = a.carry_base[c.old_carry_off + j + 1];
    }
  } else {
    const uint4 *tok = reinterpret_cast<const uint4 *>(a.tokens + c.tok_off + (u64)b0 * 16);
    const u32 q = tid & 3;
    const u64 k0 = g_lane_mult.v[4 * q], k1 = g_lane_mult.v[4 * q + 1], k2 = g_lane_mult.v[4 * q + 2],
              k3 = g_lane_mult.v[4 * q + 3];
    const u64 ksum = k0 + k1 + k2 + k3;
    uint4 v[4];
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      u32 idx = it * CHUNK + tid;
      v[it] = (idx >> 2) < nb ? __ldcs(tok + idx) : make_uint4(0, 0, 0, 0);
    }
    digest_quads(v, q, k0, k1, k2, k3, ksum, tid, nb, sd);
    __syncthreads();
    u64 cval = sd[tid];
    u64 pp = HASH_P;
#pragma unroll
    for (u32 o = 1; o < 32; o <<= 1) {
      u64 up = __shfl_up_sync(0xFFFFFFFFu, cval, o);
      if (lane >= o) cval += pp * up;
      pp *= pp;
    }
    if (lane == 31) wagg[warp] = cval;
    __syncthreads();
    u64 wc = 0;
    const u64 p32 = pp;
    for (u32 w = 0; w < warp; ++w) wc = p32 * wc + wagg[w];
    cval += g_pow_p.v[lane + 1] * wc;      // chain value of block b0 + tid with zero carry-in
    if (tid == nb - 1) sd[0] = cval;       // sd[] was consumed before the last barrier: reuse word 0 for the aggregate
    __syncthreads();
    if (warp == 0) {
      const u64 agg = sd[0];
      u64 cin;
      if (j == g0) {
        cin = g0 ? a.carry_base[c.old_carry_off + g0] : a.h0;
      } else {
        if (lane == 0) { a.agg[chunk] = agg; st_release_u32(cs.flags + chunk, 1u); }
        const u64 A = g_pow_p.v[CHUNK];    // every predecessor is a full chunk
        u64 acc_m = 1, acc_a = 0;
        int k_hi = (int)j - 1;
        bool failed = false;
        while (true) {
          const int k = k_hi - (int)lane;
          u64 m = 1, ad = 0;
          const bool mine_k = k >= (int)g0;
          const u32 idx = c.chunk_base + (u32)(mine_k ? k : 0);
          u32 f = mine_k ? 0u : 2u;   // nothing seen yet
          for (u32 it = 0; it < cs.spin_limit; ++it) {   // bounded: a limit of 0 gives up without looking
            f = mine_k ? ld_acquire_u32(cs.flags + idx) : 2u;
            if (!__any_sync(0xFFFFFFFFu, f == 0)) break;
            __nanosleep(40);
          }
          if (mine_k) {
            if (f == 2) { m = 0; ad = __ldcg(cs.incl + idx); }
            else if (f == 1) { m = A; ad = __ldcg(a.agg + idx); }
            else { m = 0; ad = 0; failed = true; }
          }
          // fold the window: lane 0 ends with M_0 o M_1 o ... o M_31 (M_31 applied first)
#pragma unroll
          for (u32 o = 1; o < 32; o <<= 1) {
            u64 m2 = __shfl_down_sync(0xFFFFFFFFu, m, o), a2 = __shfl_down_sync(0xFFFFFFFFu, ad, o);
            if (lane + o < 32) { ad = m * a2 + ad; m = m * m2; }
          }
          const u64 wm = __shfl_sync(0xFFFFFFFFu, m, 0), wa = __shfl_sync(0xFFFFFFFFu, ad, 0);
          acc_a = acc_m * wa + acc_a;
          acc_m = acc_m * wm;
          failed = __any_sync(0xFFFFFFFFu, failed);
          if (acc_m == 0 || failed) break;   // a published chain value ends the walk (A is odd: no other zero)
          k_hi -= 32;
          if (k_hi < (int)g0) { failed = true; break; }   // cannot happen: chunk g0 always publishes its chain value
        }
        if (failed && lane == 0) set_err(l.status, DERR_WAIT);
        cin = failed ? 0 : acc_a;
      }
      if (lane == 0) {
        const u64 after = g_pow_p.v[nb] * cin + agg;
        cs.incl[chunk] = after;
        st_release_u32(cs.flags + chunk, 2u);
        a.carry_base[c.carry_off + j] = cin;
        if (b0 + nb == c.n_blocks) a.carry_base[c.carry_off + j + 1] = after;   // resume point of a later call
        s_carry = cin;
      }
    }
    __syncthreads();
    if (tid < nb) {
      key = mix64(g_pow_p.v[tid + 1] * s_carry + cval);
      if (key < 2) key += 2;
    }
  }
  if (tid < nb) {
    a.keys[c.key_off + b0 + tid] = key;
    u32 ent = tab_lookup_ent(l.tab, key, l.status);
    l.b_ent[c.blk_base + b0 + tid] = ent;
    if (ent == ENT_NONE) atomicMin(&s_min, b0 + tid);
  }
  __syncthreads();
  if (tid == 0 && s_min != 0xFFFFFFFFu) atomicMin(&l.hit_len[ci], s_min);
}

// Stamps and locks the reusable prefix of every context of the batch; counts hits per tier.
struct LockArgs { Entries ent; const u32 *b_ent; const u32 *hit_len; u32 *n_hbm; u32 *n_host; u32 *n_remote; u32 now; u32 *status; };

// One CTA of CHUNK / ILP threads per 256-block chunk (the whole grid is resident at once at C4 scale with ILP = 4).
template <int ILP>
__global__ void __launch_bounds__(CHUNK / ILP) k_lock_hits(HashArgs a, LockArgs l) {
  constexpr u32 T = CHUNK / ILP;
  const u32 tid = threadIdx.x;
  dep_wait();   // before anything is read: the descriptors, the probe kernel's entry ids, prefix lengths and error word
  u32 ci;
  const HashCtx c = hash_ctx_of_chunk(a, blockIdx.x, &ci);
  // the hash / probe kernels failed: the call changes nothing. One read per CTA, so that the whole CTA agrees.
  __shared__ u32 s_err;
  __shared__ u32 s_cnt[3];
  if (tid == 0) s_err = l.status[ST_ERR];
  if (tid < 3) s_cnt[tid] = 0;
  __syncthreads();
  if (s_err) return;
  const u32 hit_len = l.hit_len[ci];
  const u32 b0 = (blockIdx.x - c.chunk_base) * CHUNK;
  u32 e[ILP];
#pragma unroll
  for (int q = 0; q < ILP; ++q) {
    const u32 b = b0 + tid + q * T;
    e[q] = b < hit_len ? l.b_ent[c.blk_base + b] : ENT_NONE;
  }
  u32 n0 = 0, n1 = 0, n2 = 0;
#pragma unroll
  for (int q = 0; q < ILP; ++q) {
    const u32 b = b0 + tid + q * T;
    if (b >= hit_len) continue;
    if (e[q] >= l.ent.n_total) { set_err(l.status, DERR_CORRUPT); continue; }
    l.ent.stamp[e[q]] = l.now;
    atomicAdd(&l.ent.infl[e[q]], 1u);
    if (e[q] < l.ent.n_hbm) ++n0; else if (e[q] < l.ent.n_hbm + l.ent.n_host) ++n1; else ++n2;
  }
  // per-tier hit counts: warp sums meet in shared memory, one global atomic per CTA and tier
  n0 = __reduce_add_sync(0xFFFFFFFFu, n0); n1 = __reduce_add_sync(0xFFFFFFFFu, n1); n2 = __reduce_add_sync(0xFFFFFFFFu, n2);
  if ((tid & 31) == 0) {
    if (n0) atomicAdd(&s_cnt[0], n0);
    if (n1) atomicAdd(&s_cnt[1], n1);
    if (n2) atomicAdd(&s_cnt[2], n2);
  }
  __syncthreads();
  if (tid == 0 && s_cnt[0]) atomicAdd(&l.n_hbm[ci], s_cnt[0]);
  if (tid == 1 && s_cnt[1]) atomicAdd(&l.n_host[ci], s_cnt[1]);
  if (tid == 2 && s_cnt[2]) atomicAdd(&l.n_remote[ci], s_cnt[2]);
}

// ======================================================================================================
// Generic ordered compaction: pred(i) for i < n -> exclusive rank among flagged items (ascending i),
// emit(i, rank) for flagged items. Three kernels: tile counts, single-CTA scan, scatter.
// ======================================================================================================
template <class Pred>
__global__ void __launch_bounds__(SCAN_TILE) k_tile_count(Pred pred, u32 n, u32 *tile_sums) {
  __shared__ u32 s;
  if (threadIdx.x == 0) s = 0;
  __syncthreads();
  u32 i = blockIdx.x * SCAN_TILE + threadIdx.x;
  bool f = i < n && pred(i);
  u32 m = __ballot_sync(0xFFFFFFFFu, f);
  if ((threadIdx.x & 31) == 0 && m) atomicAdd(&s, __popc(m));
  __syncthreads();
  if (threadIdx.x == 0) tile_sums[blockIdx.x] = s;
}

// In-place exclusive scan of tile_sums[0..n_tiles) by one CTA; total -> *total.
__global__ void __launch_bounds__(1024) k_scan_tiles(u32 *tile_sums, u32 n_tiles, u32 *total) {
  __shared__ u32 warp_sums[32];
  __shared__ u32 s_base;
  const u32 tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) s_base = 0;
  __syncthreads();
  for (u32 start = 0; start < n_tiles; start += 1024) {
    u32 i = start + tid;
    u32 v = i < n_tiles ? tile_sums[i] : 0;
    u32 x = v;
#pragma unroll
    for (u32 o = 1; o < 32; o <<= 1) { u32 y = __shfl_up_sync(0xFFFFFFFFu, x, o); if (lane >= o) x += y; }
    if (lane == 31) warp_sums[warp] = x;
    __syncthreads();
    if (warp == 0) {
      u32 w = warp_sums[lane], z = w;
#pragma unroll
      for (u32 o = 1; o < 32; o <<= 1) { u32 y = __shfl_up_sync(0xFFFFFFFFu, z, o); if (lane >= o) z += y; }
      warp_sums[lane] = z - w;  // exclusive
    }
    __syncthreads();
    u32 base = s_base;
    u32 incl = base + warp_sums[warp] + x;
    if (i < n_tiles) tile_sums[i] = incl - v;
    __syncthreads();
    if (tid == 1023) s_base = incl;
    __syncthreads();
  }
  if (tid == 0) *total = s_base;
}

template <class Pred, class Emit>
__global__ void __launch_bounds__(SCAN_TILE) k_tile_scatter(Pred pred, Emit emit, u32 n, const u32 *tile_offs) {
  __shared__ u32 warp_sums[32];
  const u32 tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  u32 i = blockIdx.x * SCAN_TILE + tid;
  bool f = i < n && pred(i);
  u32 m = __ballot_sync(0xFFFFFFFFu, f);
  if (lane == 0) warp_sums[warp] = __popc(m);
  __syncthreads();
  if (warp == 0) {
    u32 w = warp_sums[lane], z = w;
#pragma unroll
    for (u32 o = 1; o < 32; o <<= 1) { u32 y = __shfl_up_sync(0xFFFFFFFFu, z, o); if (lane >= o) z += y; }
    warp_sums[lane] = z - w;
  }
  __syncthreads();
  if (f) emit(i, tile_offs[blockIdx.x] + warp_sums[warp] + __popc(m & ((1u << lane) - 1)));
}

// ======================================================================================================
// K2: block table maintenance
// ======================================================================================================
__global__ void k_table_clear(Table t) {
  u32 i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i <= t.mask) { TSlot s; s.key = KEY_EMPTY; s.ent = ENT_NONE; s.pad = 0; t.slots[i] = s; }
}

// Re-inserts every resident entry (used after clearing, to drop tombstones).
__global__ void k_table_reinsert(Table t, Entries en, u32 *status) {
  u32 e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= en.n_total) return;
  u64 key = en.key[e];
  if (!key || is_shadow(en, e)) return;   // a clean host copy is not in the table: its block is
  u32 s = tab_find_or_claim(t, key, status);
  if (s == ENT_NONE) return;
  t.slots[s].ent = e;
  en.tslot[e] = s;
}

// ---- admission (Algorithm 1's "admit iff a slot is free", batched and deterministic) -----------------
struct AdmitCtx { u64 key_off; u32 cand_base; u32 b_start; u32 b_end; u32 res; };  // res: index of the context's result words

struct AdmitArgs {
  Table tab; Entries ent; const u64 *keys; const AdmitCtx *ctx; u32 n_ctx; u32 n_cand;
  u32 *cslot, *flag, *aux, *krank;   // per candidate scratch
  const u32 *freelist; u32 n_free;   // lowest free HBM slots, ascending; n_free = free HBM slots
  u32 *fresh; u32 fresh_base;         // list of the entries created since the mapping counts were last brought up to date
  u32 *stop;                          // per context (indexed by AdmitCtx.res)
  u32 now; u32 *status;
};
enum : u32 { CAND_OLD = 1, CAND_OWNER = 2, CAND_DUP = 3 };

__device__ __forceinline__ u32 admit_ctx_of(const AdmitArgs &a, u32 g) {
  u32 lo = 0, hi = a.n_ctx;
  while (hi - lo > 1) { u32 mid = (lo + hi) >> 1; if (a.ctx[mid].cand_base <= g) lo = mid; else hi = mid; }
  return lo;
}

// A1: every candidate finds its key or claims a slot; the lowest candidate index wins ownership.
__global__ void k_admit_claim(AdmitArgs a) {
  u32 g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= a.n_cand) return;
  const AdmitCtx c = a.ctx[admit_ctx_of(a, g)];
  u64 key = a.keys[c.key_off + c.b_start + (g - c.cand_base)];
  u32 s = tab_find_or_claim(a.tab, key, a.status);
  a.cslot[g] = s;
  if (s != ENT_NONE) atomicMin(&a.tab.slots[s].ent, CLAIM_BIT | g);  // resident ids are < CLAIM_BIT: unchanged
}

// A2: classify candidates: already resident / owner of a new key / duplicate of an earlier candidate.
__global__ void k_admit_resolve(AdmitArgs a) {
  u32 g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= a.n_cand) return;
  u32 s = a.cslot[g];
  u32 f = 0, x = 0;
  if (s != ENT_NONE) {
    u32 v = a.tab.slots[s].ent;
    if (v < CLAIM_BIT) { f = CAND_OLD; x = v; if (v >= a.ent.n_total) { set_err(a.status, DERR_CORRUPT); f = 0; } }
    else {
      x = v & ~CLAIM_BIT;
      if (x == g) f = CAND_OWNER;
      else if (x < g) f = CAND_DUP;
      else { set_err(a.status, DERR_CORRUPT); f = 0; }
    }
  }
  a.flag[g] = f;
  a.aux[g] = x;
}

struct PredOwner { const u32 *flag; __device__ bool operator()(u32 g) const { return flag[g] == CAND_OWNER; } };
struct EmitRank { u32 *krank; __device__ void operator()(u32 g, u32 r) const { krank[g] = r; } };

// A3: a context stops at its first candidate that cannot be held (the pool ran out of free slots).
__global__ void k_admit_stop(AdmitArgs a) {
  u32 g = blockIdx.x * blockDim.x + threadIdx.x;
  u32 ci = 0xFFFFFFFFu, bad = 0xFFFFFFFFu;
  if (g < a.n_cand) {
    ci = admit_ctx_of(a, g);
    const AdmitCtx c = a.ctx[ci];
    u32 f = a.flag[g];
    bool ok = f == CAND_OLD || (f == CAND_OWNER && a.krank[g] < a.n_free) ||
              (f == CAND_DUP && a.krank[a.aux[g]] < a.n_free);
    if (!ok) bad = c.b_start + (g - c.cand_base);
    ci = c.res;
  }
  // one atomic per warp when the whole warp belongs to one context (the common case)
  u32 first = __shfl_sync(0xFFFFFFFFu, ci, 0);
  if (__all_sync(0xFFFFFFFFu, ci == first)) {
    u32 m = __reduce_min_sync(0xFFFFFFFFu, bad);
    if ((threadIdx.x & 31) == 0 && m != 0xFFFFFFFFu && first != 0xFFFFFFFFu) atomicMin(&a.stop[first], m);
  } else if (bad != 0xFFFFFFFFu) {
    atomicMin(&a.stop[ci], bad);
  }
}

// A4: apply. Held candidates stamp/lock their block; owners that got a slot create the entry; owners
// beyond the stop point give their claimed table slot back as a tombstone.
__global__ void k_admit_apply(AdmitArgs a) {
  u32 g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= a.n_cand) return;
  if (a.status[ST_ERR]) return;
  const AdmitCtx c = a.ctx[admit_ctx_of(a, g)];
  u32 b = c.b_start + (g - c.cand_base);
  u32 f = a.flag[g];
  bool held = b < a.stop[c.res];
  if (f == CAND_OLD) {
    if (held) { u32 e = a.aux[g]; a.ent.stamp[e] = a.now; atomicAdd(&a.ent.infl[e], 1u); atomicAdd(&a.status[ST_ADOPTED], 1u); }
  } else if (f == CAND_OWNER) {
    u32 s = a.cslot[g];
    if (held) {
      KVT_CHECK(a.krank[g] < a.n_free, a.status, return);
      u32 e = a.freelist[a.krank[g]];
      KVT_CHECK(e < a.ent.n_hbm && a.ent.key[e] == 0 && s <= a.tab.mask, a.status, return);
      a.ent.key[e] = a.keys[c.key_off + b];
      a.ent.stamp[e] = a.now; a.ent.depth[e] = b; a.ent.cnt[e] = 0; a.ent.floor[e] = 0; a.ent.tslot[e] = s; a.ent.link[e] = ENT_NONE;
      atomicAdd(&a.ent.infl[e], 1u);
      a.tab.slots[s].ent = e;
      a.fresh[a.fresh_base + atomicAdd(&a.status[ST_INSERTED], 1u)] = e;
    } else {
      a.tab.slots[s].key = KEY_TOMB;
      a.tab.slots[s].ent = ENT_NONE;
      atomicAdd(&a.status[ST_TOMBS], 1u);
    }
  } else if (f == CAND_DUP) {
    if (held) { u32 e = a.freelist[a.krank[a.aux[g]]]; atomicAdd(&a.ent.infl[e], 1u); atomicAdd(&a.status[ST_ADOPTED], 1u); }
  }
}

// ---- per-context helpers -------------------------------------------------------------------------------
// Releases the in-flight locks of blocks [0, n) of a key list (prefill done / terminate).
__global__ void k_unlock(Table t, Entries en, const u64 *keys, u32 n, u32 now, u32 do_stamp, u32 *status) {
  u32 b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= n) return;
  u32 e = tab_lookup_ent(t, keys[b], status);
  if (e >= en.n_total) { set_err(status, DERR_CORRUPT); return; }
  u32 old = atomicSub(&en.infl[e], 1u);
  if (old == 0) { atomicAdd(&en.infl[e], 1u); set_err(status, DERR_CORRUPT); }
  if (do_stamp) en.stamp[e] = now;
}

// Residency of every key of a list (block map).
__global__ void k_block_map(Table t, Entries en, const u64 *keys, u32 n, u8 *tier, u32 *slot, u32 *status) {
  u32 b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= n) return;
  u32 e = tab_lookup_ent(t, keys[b], status);
  if (e >= en.n_total) { tier[b] = 0xFF; slot[b] = 0xFFFFFFFFu; }
  else if (e < en.n_hbm) { tier[b] = 0; slot[b] = e; }
  else if (e < en.n_hbm + en.n_host) { tier[b] = 1; slot[b] = e - en.n_hbm; }
  else { tier[b] = 2; slot[b] = e - en.n_hbm - en.n_host; }
}

// ======================================================================================================
// K3: classifier (Section 6.1). The engine keeps, per resident block, how many (context, block) mappings of each
// rank point at its key (Entries.cnt); the block's state is read off those counts. A mapping's rank is the highest
// message rank over the messages whose token span touches the block. The counts are updated by events, not
// recomputed: for every context whose messages, mapped prefix or key list changed since it was last accounted
// for, one thread per block takes the old contribution away and adds the new one (k_map_delta); keys that entered
// the table since then receive the contributions of every context that already mapped them (k_run_filter /
// k_run_fixup). The full recomputation is the same delta kernel run from zero counts over all contexts.
// ======================================================================================================
struct MsgTables { const u32 *start, *end; const u8 *rank; };   // message spans of all accounted-for contexts, by offset

// Rank of block b under a message table slice [off, off + n): highest rank over the messages touching tokens [16 b, 16 b + 16).
__device__ __forceinline__ u32 block_rank(const MsgTables &t, u32 off, u32 n, u32 b) {
  const u32 t0 = b * 16, t1 = t0 + 16;
  const u32 *ms = t.start + off, *me = t.end + off;
  const u8 *mr = t.rank + off;
  u32 l = 0, h = n;   // first message whose end is beyond t0 (ends are non-decreasing)
  while (l < h) { const u32 mid = (l + h) >> 1; if (me[mid] > t0) h = mid; else l = mid + 1; }
  u32 r = 0;
  for (u32 j = l; j < n && ms[j] < t1; ++j)
    if (me[j] > ms[j] && mr[j] > r) r = mr[j];
  return r;
}

// One context of a delta pass: what was accounted for (old) and what holds now (new).
struct DeltaCtx {
  u64 old_key_off, new_key_off;        // key lists (u64 index into keys)
  u32 old_valid, new_valid;            // mapped prefix lengths
  u32 old_tbl, old_n, new_tbl, new_n;  // message table slices
  u32 map_base;                        // first item of this context in the flattened (context, block) index space
  u32 pad;
};
struct DeltaArgs {
  Table tab; Entries ent; const u64 *keys; const DeltaCtx *ctx; u32 n_ctx; u32 n_map;
  MsgTables tbl; u32 *status;
  u32 *first_miss;   // per listed context: index of its first non-resident block; nullptr = orphans keep their state
};

// Context that owns item g (the last one whose map_base is <= g). Every thread of the CTA calls it: the
// bases are staged in shared memory by one round of loads when they fit.
constexpr u32 CTX_STAGE = 1024;
__device__ __forceinline__ u32 delta_ctx_of_item(const DeltaArgs &a, u32 g) {
  __shared__ u32 s_base[CTX_STAGE];
  const bool staged = a.n_ctx <= CTX_STAGE;
  if (staged) {
    for (u32 t = threadIdx.x; t < a.n_ctx; t += blockDim.x) s_base[t] = a.ctx[t].map_base;
    __syncthreads();
  }
  u32 lo = 0, hi = a.n_ctx;
  while (hi - lo > 1) {
    u32 mid = (lo + hi) >> 1;
    if ((staged ? s_base[mid] : a.ctx[mid].map_base) <= g) lo = mid; else hi = mid;
  }
  return lo;
}

// Reachability pre-pass of the full recomputation: the first block of every context's mapped prefix that is resident
// in no tier. A lookup stops there, so the blocks behind it cannot be reused through this context.
__global__ void k_first_miss(DeltaArgs a) {
  u32 g = blockIdx.x * blockDim.x + threadIdx.x;
  const u32 lo = delta_ctx_of_item(a, g);
  if (g >= a.n_map) return;
  const DeltaCtx c = a.ctx[lo];
  const u32 b = g - c.map_base;
  if (b >= c.new_valid) return;
  if (tab_lookup_ent(a.tab, a.keys[c.new_key_off + b], a.status) == ENT_NONE) atomicMin(&a.first_miss[lo], b);
}

__device__ __forceinline__ void cnt_add(const DeltaArgs &a, u64 key, u64 delta) {
  const u32 e = tab_lookup_ent(a.tab, key, a.status);   // ENT_NONE: mapped but not resident
  KVT_CHECK(e == ENT_NONE || (e < a.ent.n_total && a.ent.key[e] == key), a.status, return);
  if (e < a.ent.n_total) atomicAdd((unsigned long long *)&a.ent.cnt[e], (unsigned long long)delta);
}

__global__ void k_map_delta(DeltaArgs a) {
  u32 g = blockIdx.x * blockDim.x + threadIdx.x;
  const u32 lo = delta_ctx_of_item(a, g);
  if (g >= a.n_map) return;
  const DeltaCtx c = a.ctx[lo];
  const u32 b = g - c.map_base;
  const bool has_old = b < c.old_valid, has_new = b < c.new_valid && !(a.first_miss && b >= a.first_miss[lo]);
  const u64 k_old = has_old ? a.keys[c.old_key_off + b] : 0, k_new = has_new ? a.keys[c.new_key_off + b] : 0;
  const u32 r_old = has_old ? block_rank(a.tbl, c.old_tbl, c.old_n, b) : 0;
  const u32 r_new = has_new ? block_rank(a.tbl, c.new_tbl, c.new_n, b) : 0;
  if (k_old == k_new) {
    if (r_old != r_new && k_new) cnt_add(a, k_new, cnt_unit(r_new) - cnt_unit(r_old));
  } else {
    if (r_old) cnt_add(a, k_old, 0ull - cnt_unit(r_old));
    if (r_new) cnt_add(a, k_new, cnt_unit(r_new));
  }
}

// Entries created since the counts were last brought up to date start at zero. Each of them receives, once, the
// contribution of every accounted-for mapping (snapshot) whose key at the entry's chain depth is the entry's key.
// Between two such passes entries are neither moved nor dropped, so the list holds valid, distinct entry ids.
struct SnapDesc { u64 key_off; u32 valid, tbl, n, pad; };
struct FixArgs {
  Table tab; Entries ent; const u64 *keys; const SnapDesc *snaps; u32 n_snaps;
  MsgTables tbl; const u32 *fresh; u32 n_fresh; u32 *status;
};

__global__ void k_fresh_fixup(FixArgs a) {
  const u32 i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= a.n_fresh) return;
  const u32 e = a.fresh[i];
  if (e >= a.ent.n_total) { set_err(a.status, DERR_CORRUPT); return; }
  const u64 key = a.ent.key[e];
  const u32 d = a.ent.depth[e];
  u64 sum = 0;
  for (u32 q = 0; q < a.n_snaps; ++q) {
    const SnapDesc sn = a.snaps[q];
    if (d < sn.valid && a.keys[sn.key_off + d] == key) sum += cnt_unit(block_rank(a.tbl, sn.tbl, sn.n, d));
  }
  if (sum) a.ent.cnt[e] += sum;   // nobody else touches this entry in this kernel
}

// Cross-check of the event-driven counts against a full recomputation (debug mode): any difference is an error.
__global__ void k_cnt_compare(const u64 *a, const u64 *b, u32 n, u32 *status) {
  const u32 e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e < n && a[e] != b[e]) set_err(status, DERR_CORRUPT);
}

// ======================================================================================================
// K4: victim selection (Algorithm 1 order; Section 6.2 recency). Candidates of a tier: resident, not in
// flight, rank <= max_rank (2, or 3 when the incoming KV is Pinned). The order is the ascending order of the
// composite (packed key, slot), packed key = [copy bit] rank | recency | inverted depth. The first k of that
// order are found without sorting the tier:
//   keys    : one pass over the tier writes every slot's packed key and counts the composite's top digit;
//   level l : MSB-first radix select. Each level kernel first turns the previous level's histogram into the bin
//             in which the k-th smallest composite lies (every CTA does this small scan itself, so no kernel
//             waits for another), then counts the next digit of the slots inside that bin. The search stops as
//             soon as the bin holds at most SEL_SLACK slots; the composite is unique per slot, so the last
//             level always ends it;
//   gather  : the slots below the bin (all selected) and the slots of the bin go into the pair list in slot
//             order (per-CTA counts, then every CTA adds up the counts before it): k <= M <= k + SEL_SLACK pairs;
//   sort    : stable LSD radix sort of those M pairs on the key bits, 10 bits per pass; ties end slot-ascending;
//   emit    : the first k pairs, with their states.
// Every kernel reads its arguments from one record in device memory, so the whole sequence is a fixed CUDA graph
// per (tier, level count, pass count) and a call is one upload and one graph launch. Work scales with k, not with
// the number of candidates.
// ======================================================================================================
typedef unsigned __int128 u128;
constexpr u32 SEL_W0 = 11, SEL_WN = 13;            // digit widths of level 0 and of the later levels
constexpr u32 SEL_BINS = 1u << SEL_WN;            // bins of a histogram (level 0 uses the first 2^11)
constexpr u32 SEL_SLACK = 4096;                   // a boundary bin this small ends the search
constexpr u32 SEL_MAX_LEVELS = 9;                 // 11 + 8 * 13 = 115 bits >= 63 key bits + 31 slot bits
constexpr u32 SEL_ITEMS = 4, SEL_CTA = 1024;      // slots per thread / threads per CTA of the tier-wide passes
constexpr u32 SEL_TILE = SEL_ITEMS * SEL_CTA;     // slots per CTA
constexpr u64 SEL_NOT_KEY = ~0ull;                // packed key of a slot that is not a candidate (real keys have bit 63 clear)
constexpr u32 RADIX_BITS = 10, RADIX_BINS = 1u << RADIX_BITS;
constexpr u32 SORT_TILE = 1024;                   // pairs per CTA in the radix-sort kernels (8 warps x 128)
constexpr int SORT_ITERS = SORT_TILE / 256;       // pairs per thread

struct SelState { u32 done, need, below, lo; u32 pfx[4]; };   // after the boundaries of levels 0 .. j-1
struct SelArgs {
  Entries ent; u32 e0, n_slots;       // entry range of the tier
  u32 n_req; u32 now; u32 stamp_bits, depth_bits; u32 mru; u32 max_rank; u32 one_tier;
  u32 copy_bit;                       // 1: the key carries a leading "resident block" bit (host tier with clean copies)
  u32 slot_bits;                      // bits of a slot number; the composite is (key << slot_bits) | slot
  u32 n_levels; u8 lev_lo[SEL_MAX_LEVELS], lev_w[SEL_MAX_LEVELS];   // level l looks at composite bits [lo, lo + w)
  u64 *slot_key;                      // per slot of the tier: packed key or SEL_NOT_KEY
  u32 *hist;                          // n_levels x SEL_BINS counters, zero at the start of a call
  SelState *state;                    // n_levels + 1 records; record 0 is unused
  u32 *cta_count;                     // per CTA of the tier-wide passes: slots it contributes to the gathered set
  u64 *pair_key; u32 *pair_val;       // gathered pairs
  u32 n_emit, rank_shift; u32 *slots_out; u8 *states_out;   // victim list
  u32 *status;
};

// The argument record of a call, staged once per CTA in shared memory (a per-thread copy would land in local
// memory, because the level tables are indexed at run time).
__device__ __forceinline__ const SelArgs &sel_args(const SelArgs *pa) {
  __shared__ SelArgs s_args;
  const u32 *src = reinterpret_cast<const u32 *>(pa);
  u32 *dst = reinterpret_cast<u32 *>(&s_args);
  for (u32 i = threadIdx.x; i < sizeof(SelArgs) / 4; i += blockDim.x) dst[i] = __ldg(src + i);
  __syncthreads();
  return s_args;
}

__device__ __forceinline__ u128 sel_comp(const SelArgs &a, u64 key, u32 slot) { return ((u128)key << a.slot_bits) | slot; }
__device__ __forceinline__ u128 sel_prefix(const SelState &s) {
  return ((u128)(((u64)s.pfx[3] << 32) | s.pfx[2]) << 64) | (((u64)s.pfx[1] << 32) | s.pfx[0]);
}

// Adds one to bin d of the CTA's shared histogram for every lane with ok set. A warp whose lanes all hold the same
// digit (pools with few distinct stamps) adds once; otherwise every lane adds for itself.
__device__ __forceinline__ void sel_count_digit(u32 *h, bool ok, u32 d) {
  int same = 0;
  __match_all_sync(0xFFFFFFFFu, ok ? d : 0xFFFFFFFFu, &same);
  if (same) { if (ok && (threadIdx.x & 31) == 0) atomicAdd(&h[d], 32u); }
  else if (ok) atomicAdd(&h[d], 1u);
}

__device__ __forceinline__ void sel_flush_hist(const u32 *h, u32 bins, u32 *ghist) {
  for (u32 b = threadIdx.x; b < bins; b += SEL_CTA) { const u32 v = h[b]; if (v) atomicAdd(&ghist[b], v); }
}

// Every thread of a SEL_CTA-thread CTA calls this. Applies the boundary of level `lev` (its histogram is complete:
// it was written by an earlier kernel) to the state before it and returns the state after it. The state says which
// composite prefix still has to be searched (pfx, above bit lo), how many of the wanted slots lie in it (need) and
// how many candidates lie below it (below); done ends the search: every candidate whose composite, shifted right
// by lo, is <= pfx belongs to the gathered set.
__device__ SelState sel_apply_level(const SelArgs &a, u32 lev, SelState in) {
  __shared__ u32 s_warp[32];
  __shared__ SelState s_out;
  if (in.done) return in;
  const u32 tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const u32 bins = 1u << a.lev_w[lev];
  const u32 per = (bins + SEL_CTA - 1) / SEL_CTA;   // consecutive bins per thread (<= 8)
  const u32 *h = a.hist + (u64)lev * SEL_BINS;
  u32 mine = 0;
  for (u32 q = 0; q < per; ++q) { const u32 b = tid * per + q; if (b < bins) mine += h[b]; }
  u32 x = mine;
#pragma unroll
  for (u32 o = 1; o < 32; o <<= 1) { u32 y = __shfl_up_sync(0xFFFFFFFFu, x, o); if (lane >= o) x += y; }
  if (lane == 31) s_warp[warp] = x;
  __syncthreads();
  if (warp == 0) {
    u32 w = s_warp[lane], z = w;
#pragma unroll
    for (u32 o = 1; o < 32; o <<= 1) { u32 y = __shfl_up_sync(0xFFFFFFFFu, z, o); if (lane >= o) z += y; }
    s_warp[lane] = z - w;
    if (lane == 31) {   // all candidates of this level: fewer than wanted means "take everything"
      const u32 total = z;
      if (lev == 0) a.status[ST_TOTAL] = total;   // same value from every CTA
      if (total < in.need || total == 0) {
        SelState o = in;
        o.done = 1; o.below = in.below + total; o.need = 0; o.lo = 0;
        o.pfx[0] = o.pfx[1] = o.pfx[2] = o.pfx[3] = 0xFFFFFFFFu;   // every composite is below this
        a.status[ST_AUX] = o.below;                                  // size of the gathered set
        s_out = o;
      } else {
        s_out.done = 2;   // marker: a bin will be found below
      }
    }
  }
  __syncthreads();
  const bool take_all = s_out.done == 1;
  const u32 before = s_warp[warp] + x - mine;   // candidates in the bins of earlier threads
  __syncthreads();
  if (!take_all && before < in.need && in.need <= before + mine) {   // exactly one thread
    u32 cum = before;
    for (u32 q = 0; q < per; ++q) {
      const u32 b = tid * per + q;
      const u32 c = b < bins ? h[b] : 0;
      if (in.need <= cum + c) {
        SelState o;
        const u128 p = (sel_prefix(in) << a.lev_w[lev]) | b;
        o.pfx[0] = (u32)p; o.pfx[1] = (u32)(p >> 32); o.pfx[2] = (u32)(p >> 64); o.pfx[3] = (u32)(p >> 96);
        o.below = in.below + cum;
        o.need = in.need - cum;
        o.lo = a.lev_lo[lev];
        o.done = (c <= SEL_SLACK || lev + 1 == a.n_levels) ? 1u : 0u;
        if (o.done) a.status[ST_AUX] = o.below + c;   // size of the gathered set (same value from every CTA)
        s_out = o;
        break;
      }
      cum += c;
    }
  }
  __syncthreads();
  SelState out = s_out;
  __syncthreads();
  return out;
}

__device__ __forceinline__ SelState sel_initial(const SelArgs &a) {
  SelState in;
  in.done = 0; in.need = a.n_req; in.below = 0; in.lo = 0; in.pfx[0] = in.pfx[1] = in.pfx[2] = in.pfx[3] = 0;
  return in;
}

// Pass over the tier: packed key of every slot, histogram of the composite's top digit. All fields of the SEL_ITEMS
// slots of a thread are fetched before any of them is looked at, so the loads are in flight together.
__global__ void __launch_bounds__(SEL_CTA) k_sel_keys(const SelArgs *pa) {
  __shared__ u32 h[1u << SEL_W0];
  const SelArgs &a = sel_args(pa);
  for (u32 b = threadIdx.x; b < (1u << SEL_W0); b += SEL_CTA) h[b] = 0;
  const u32 lo = a.lev_lo[0], mask = (1u << a.lev_w[0]) - 1;
  u64 ekey[SEL_ITEMS];
  u32 link[SEL_ITEMS], infl[SEL_ITEMS], rank[SEL_ITEMS], stamp[SEL_ITEMS], depth[SEL_ITEMS];
#pragma unroll
  for (u32 it = 0; it < SEL_ITEMS; ++it) {
    const u32 i = (blockIdx.x * SEL_ITEMS + it) * SEL_CTA + threadIdx.x;
    const u32 e = a.e0 + min(i, a.n_slots - 1);
    ekey[it] = a.ent.key[e]; link[it] = a.ent.link[e]; infl[it] = a.ent.infl[e]; rank[it] = entry_rank(a.ent, e);
    stamp[it] = a.ent.stamp[e]; depth[it] = a.ent.depth[e];
  }
  __syncthreads();
#pragma unroll
  for (u32 it = 0; it < SEL_ITEMS; ++it) {
    const u32 i = (blockIdx.x * SEL_ITEMS + it) * SEL_CTA + threadIdx.x;
    bool ok = false;
    u32 d = 0;
    if (i < a.n_slots) {
      const bool sh = a.e0 + i >= a.ent.n_hbm && link[it] != ENT_NONE;       // clean host copy of an HBM block
      const u32 r = a.one_tier ? 1u : rank[it];
      u64 key = SEL_NOT_KEY;
      if (ekey[it] && (sh || (!infl[it] && r <= a.max_rank))) {
        const u64 rr = sh ? 0u : r;
        const u64 rec = (rr == 1 && a.mru && !sh) ? (u64)a.now - stamp[it] : (u64)stamp[it];   // newest first inside the idle tier
        const u64 dinv = ((1ull << a.depth_bits) - 1) - depth[it];                              // chain tail first
        key = (a.copy_bit ? (u64)(sh ? 0u : 1u) << (2 + a.stamp_bits + a.depth_bits) : 0) |    // copies before resident blocks
              (rr << (a.stamp_bits + a.depth_bits)) | (rec << a.depth_bits) | dinv;
        ok = true;
        d = (u32)(sel_comp(a, key, i) >> lo) & mask;
      }
      a.slot_key[i] = key;
    }
    sel_count_digit(h, ok, d);
  }
  __syncthreads();
  sel_flush_hist(h, 1u << a.lev_w[0], a.hist);
}

// Level lev >= 1: boundary of level lev - 1, then the histogram of digit lev inside the boundary bin.
__global__ void __launch_bounds__(SEL_CTA) k_sel_level(const SelArgs *pa, u32 lev) {
  __shared__ u32 h[SEL_BINS];
  const SelArgs &a = sel_args(pa);
  if (lev >= a.n_levels) return;
  const SelState st = sel_apply_level(a, lev - 1, lev == 1 ? sel_initial(a) : a.state[lev - 1]);
  if (blockIdx.x == 0 && threadIdx.x == 0) a.state[lev] = st;
  if (st.done) return;
  const u32 bins = 1u << a.lev_w[lev];
  for (u32 b = threadIdx.x; b < bins; b += SEL_CTA) h[b] = 0;
  __syncthreads();
  const u128 pfx = sel_prefix(st);
  const u32 lo = a.lev_lo[lev], mask = bins - 1;
  bool any = false;
#pragma unroll
  for (u32 it = 0; it < SEL_ITEMS; ++it) {
    const u32 i = (blockIdx.x * SEL_ITEMS + it) * SEL_CTA + threadIdx.x;
    bool ok = false;
    u32 d = 0;
    if (i < a.n_slots) {
      const u64 key = a.slot_key[i];
      if (key != SEL_NOT_KEY) {
        const u128 c = sel_comp(a, key, i);
        if ((c >> st.lo) == pfx) { ok = true; d = (u32)(c >> lo) & mask; }
      }
    }
    sel_count_digit(h, ok, d);
    any = any || ok;
  }
  if (__syncthreads_or(any)) sel_flush_hist(h, bins, a.hist + (u64)lev * SEL_BINS);
}

// Last boundary, then how many slots of every CTA's stretch belong to the gathered set (every candidate whose
// composite prefix is at or below the boundary bin).
__global__ void __launch_bounds__(SEL_CTA) k_sel_count(const SelArgs *pa) {
  __shared__ u32 s_cnt;
  const SelArgs &a = sel_args(pa);
  const SelState st = sel_apply_level(a, a.n_levels - 1, a.n_levels == 1 ? sel_initial(a) : a.state[a.n_levels - 1]);
  if (blockIdx.x == 0 && threadIdx.x == 0) a.state[a.n_levels] = st;   // always done: the last level's bins hold one slot each
  if (threadIdx.x == 0) s_cnt = 0;
  __syncthreads();
  const u128 pfx = sel_prefix(st);
  u32 mine = 0;
#pragma unroll
  for (u32 it = 0; it < SEL_ITEMS; ++it) {
    const u32 i = (blockIdx.x * SEL_ITEMS + it) * SEL_CTA + threadIdx.x;
    const u64 key = i < a.n_slots ? a.slot_key[i] : SEL_NOT_KEY;
    mine += key != SEL_NOT_KEY && (sel_comp(a, key, i) >> st.lo) <= pfx;
  }
  mine = __reduce_add_sync(0xFFFFFFFFu, mine);
  if ((threadIdx.x & 31) == 0 && mine) atomicAdd(&s_cnt, mine);
  __syncthreads();
  if (threadIdx.x == 0) a.cta_count[blockIdx.x] = s_cnt;
}

// The gathered set in slot order: a CTA's first pair goes behind the pairs of all CTAs before it.
__global__ void __launch_bounds__(SEL_CTA) k_sel_gather(const SelArgs *pa) {
  __shared__ u32 s_warp[SEL_ITEMS][32];   // pairs per (iteration, warp), then their exclusive prefix in slot order
  __shared__ u32 s_red[32];
  const SelArgs &a = sel_args(pa);
  const SelState st = a.state[a.n_levels];
  const u128 pfx = sel_prefix(st);
  const u32 tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  u32 before = 0;   // pairs of the CTAs before this one
  for (u32 c = tid; c < blockIdx.x; c += SEL_CTA) before += a.cta_count[c];
  before = __reduce_add_sync(0xFFFFFFFFu, before);
  if (lane == 0) s_red[warp] = before;
  u64 key[SEL_ITEMS];
  u32 m[SEL_ITEMS];
#pragma unroll
  for (u32 it = 0; it < SEL_ITEMS; ++it) {
    const u32 i = (blockIdx.x * SEL_ITEMS + it) * SEL_CTA + tid;
    key[it] = i < a.n_slots ? a.slot_key[i] : SEL_NOT_KEY;
    const bool in_set = key[it] != SEL_NOT_KEY && (sel_comp(a, key[it], i) >> st.lo) <= pfx;
    m[it] = __ballot_sync(0xFFFFFFFFu, in_set);
    if (lane == 0) s_warp[it][warp] = __popc(m[it]);
  }
  __syncthreads();
  if (warp == 0) {
    u32 base = s_red[lane];
#pragma unroll
    for (u32 o = 16; o > 0; o >>= 1) base += __shfl_xor_sync(0xFFFFFFFFu, base, o);
    // exclusive scan over (iteration, warp) in that order = ascending slot
    u32 run = base;
#pragma unroll
    for (u32 it = 0; it < SEL_ITEMS; ++it) {
      const u32 w = s_warp[it][lane];
      u32 z = w;
#pragma unroll
      for (u32 o = 1; o < 32; o <<= 1) { u32 y = __shfl_up_sync(0xFFFFFFFFu, z, o); if (lane >= o) z += y; }
      s_warp[it][lane] = run + z - w;
      run += __shfl_sync(0xFFFFFFFFu, z, 31);
    }
    if (blockIdx.x == gridDim.x - 1 && lane == 0) a.status[ST_M] = run;   // size of the gathered set
  }
  __syncthreads();
#pragma unroll
  for (u32 it = 0; it < SEL_ITEMS; ++it) {
    if (!((m[it] >> lane) & 1)) continue;
    const u32 i = (blockIdx.x * SEL_ITEMS + it) * SEL_CTA + tid;
    const u32 p = s_warp[it][warp] + __popc(m[it] & ((1u << lane) - 1));
    if (p >= a.n_slots) { set_err(a.status, DERR_CORRUPT); continue; }   // cannot happen: at most one pair per slot
    a.pair_key[p] = key[it];
    a.pair_val[p] = i;
  }
}

// ---- stable LSD radix sort, RADIX_BITS per pass; element count read from the status block ----------------
__global__ void __launch_bounds__(256) k_radix_hist(const u64 *keys, const u32 *status, u32 shift, u32 *counts) {
  __shared__ u32 h[RADIX_BINS];
  const u32 m = status[ST_M];
  const u32 n_tiles = (m + SORT_TILE - 1) / SORT_TILE;
  if (blockIdx.x >= n_tiles) return;
  for (u32 d = threadIdx.x; d < RADIX_BINS; d += 256) h[d] = 0;
  __syncthreads();
  const u32 base = blockIdx.x * SORT_TILE + threadIdx.x;
  u64 kreg[SORT_ITERS];
#pragma unroll
  for (int it = 0; it < SORT_ITERS; ++it) kreg[it] = base + it * 256 < m ? keys[base + it * 256] : 0;   // loads first, then the atomics
#pragma unroll
  for (int it = 0; it < SORT_ITERS; ++it)
    if (base + it * 256 < m) atomicAdd(&h[(u32)(kreg[it] >> shift) & (RADIX_BINS - 1)], 1u);
  __syncthreads();
  for (u32 d = threadIdx.x; d < RADIX_BINS; d += 256) counts[d * n_tiles + blockIdx.x] = h[d];   // digit-major
}

// One warp per digit: exclusive scan of that digit's per-tile counts in place, digit total to row_total.
__global__ void __launch_bounds__(256) k_radix_scan(u32 *counts, u32 *row_total, const u32 *status) {
  const u32 m = status[ST_M];
  const u32 n_tiles = (m + SORT_TILE - 1) / SORT_TILE;
  const u32 lane = threadIdx.x & 31, d = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (d >= RADIX_BINS) return;
  u32 *row = counts + d * n_tiles;
  u32 run = 0;
  for (u32 t0 = 0; t0 < n_tiles; t0 += 32) {
    u32 t = t0 + lane;
    u32 v = t < n_tiles ? row[t] : 0, x = v;
#pragma unroll
    for (u32 o = 1; o < 32; o <<= 1) { u32 y = __shfl_up_sync(0xFFFFFFFFu, x, o); if (lane >= o) x += y; }
    if (t < n_tiles) row[t] = run + x - v;
    run += __shfl_sync(0xFFFFFFFFu, x, 31);
  }
  if (lane == 0) row_total[d] = run;
}

__global__ void __launch_bounds__(256) k_radix_scatter(const u64 *keys_in, const u32 *vals_in, u64 *keys_out, u32 *vals_out,
                                                       const u32 *status, u32 shift, const u32 *offsets, const u32 *row_total) {
  // each warp owns SORT_TILE / 8 consecutive items of the tile and walks them in order, so equal digits keep
  // their input order (stable)
  __shared__ u32 cnt[8][RADIX_BINS];
  __shared__ u32 dbase[RADIX_BINS];
  __shared__ u32 wsum[8];
  constexpr u32 DPT = RADIX_BINS / 256;   // digits per thread in the digit scans
  const u32 m = status[ST_M];
  const u32 n_tiles = (m + SORT_TILE - 1) / SORT_TILE;
  if (blockIdx.x >= n_tiles) return;
  const u32 tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (u32 k = tid; k < 8 * RADIX_BINS; k += 256) (&cnt[0][0])[k] = 0;
  __syncthreads();
  const u32 base = blockIdx.x * SORT_TILE + warp * (SORT_TILE / 8);
  u64 kreg[SORT_ITERS];
  u32 vreg[SORT_ITERS];
#pragma unroll
  for (int it = 0; it < SORT_ITERS; ++it) {   // all loads first: the ranking loop below synchronises the warp in every step
    u32 i = base + it * 32 + lane;
    kreg[it] = i < m ? keys_in[i] : 0;
    vreg[it] = i < m ? vals_in[i] : 0;
  }
#pragma unroll
  for (int it = 0; it < SORT_ITERS; ++it) {
    u32 i = base + it * 32 + lane;
    bool ok = i < m;
    u32 d = (u32)(kreg[it] >> shift) & (RADIX_BINS - 1);
    u32 peers = __match_any_sync(0xFFFFFFFFu, ok ? d : RADIX_BINS);
    if (ok && (peers & ((1u << lane) - 1)) == 0) cnt[warp][d] += __popc(peers);
    __syncwarp();
  }
  __syncthreads();
  {  // first position of every digit = exclusive scan of the digit totals (DPT consecutive digits per thread)
    u32 v[DPT], sum = 0;
#pragma unroll
    for (u32 q = 0; q < DPT; ++q) { v[q] = row_total[tid * DPT + q]; sum += v[q]; }
    u32 x = sum;
#pragma unroll
    for (u32 o = 1; o < 32; o <<= 1) { u32 y = __shfl_up_sync(0xFFFFFFFFu, x, o); if (lane >= o) x += y; }
    if (lane == 31) wsum[warp] = x;
    __syncthreads();
    u32 run = x - sum;
    for (u32 w = 0; w < warp; ++w) run += wsum[w];
#pragma unroll
    for (u32 q = 0; q < DPT; ++q) { dbase[tid * DPT + q] = run; run += v[q]; }
  }
  __syncthreads();
  for (u32 d = tid; d < RADIX_BINS; d += 256) {   // per digit: exclusive scan across the 8 warps, plus the tile's offset inside the digit
    u32 run = dbase[d] + offsets[d * n_tiles + blockIdx.x];
#pragma unroll
    for (int w = 0; w < 8; ++w) { u32 c = cnt[w][d]; cnt[w][d] = run; run += c; }
  }
  __syncthreads();
#pragma unroll
  for (int it = 0; it < SORT_ITERS; ++it) {
    u32 i = base + it * 32 + lane;
    bool ok = i < m;
    u32 d = (u32)(kreg[it] >> shift) & (RADIX_BINS - 1);
    u32 peers = __match_any_sync(0xFFFFFFFFu, ok ? d : RADIX_BINS);
    u32 before = __popc(peers & ((1u << lane) - 1));
    u32 pos = 0;
    if (ok) pos = cnt[warp][d] + before;
    __syncwarp();
    if (ok && before == 0) cnt[warp][d] += __popc(peers);
    __syncwarp();
    KVT_CHECK(!ok || pos < m, const_cast<u32 *>(status), continue);
    if (ok) { keys_out[pos] = kreg[it]; vals_out[pos] = vreg[it]; }
  }
}

// Victim list for the caller: slot, and its state: the rank, | 0x80 for an HBM block that still has a clean host
// copy (moving it out needs no copy), or 0xFE for a host slot that is such a copy.
__global__ void k_sel_emit(const SelArgs *pa, const u64 *keys, const u32 *vals) {
  const SelArgs &a = sel_args(pa);
  const u32 n = min(a.n_emit, a.status[ST_M]);   // only the first ST_M pairs exist
  // four victims per thread: the list usually goes over the host link, where one 16-byte and one 4-byte store per
  // thread travel better than four 4-byte and four single-byte ones
  const bool wide = !((uintptr_t)a.slots_out & 15) && !((uintptr_t)a.states_out & 3);
  for (u32 i0 = (blockIdx.x * blockDim.x + threadIdx.x) * 4; i0 < n; i0 += gridDim.x * blockDim.x * 4) {
    u32 slot[4];
    u8 st[4];
    bool all = true;
#pragma unroll
    for (u32 j = 0; j < 4; ++j) {
      const u32 i = i0 + j;
      slot[j] = i < n ? vals[i] : 0xFFFFFFFFu;
      st[j] = 0;
      if (slot[j] >= a.n_slots) { all = false; continue; }
      const u64 k = keys[i] >> a.rank_shift;
      const bool primary = a.copy_bit ? (k >> 2) & 1 : true;
      const u32 link = a.ent.link[a.e0 + slot[j]];
      st[j] = !primary ? (u8)0xFE : (u8)((k & 3) | (link != ENT_NONE ? 0x80 : 0));
    }
    if (wide && all) {
      *reinterpret_cast<uint4 *>(a.slots_out + i0) = make_uint4(slot[0], slot[1], slot[2], slot[3]);
      *reinterpret_cast<uchar4 *>(a.states_out + i0) = make_uchar4(st[0], st[1], st[2], st[3]);
    } else {
#pragma unroll
      for (u32 j = 0; j < 4; ++j)
        if (slot[j] < a.n_slots) { a.slots_out[i0 + j] = slot[j]; a.states_out[i0 + j] = st[j]; }
    }
  }
}

// ======================================================================================================
// Slot-list operations (offload / reload / release / compact): validate, plan, apply.
// ======================================================================================================
struct ListArgs {
  Table tab; Entries ent;
  const u32 *ids; u32 n; u32 e0, n_slots;   // listed slots of the source tier (entry = e0 + id)
  u32 dst_e0;                                // first entry id of the destination tier
  u32 *live;                                 // per item: LIST_DROP, LIST_COPY (needs a free destination slot), LIST_CLEAN
  u32 *lidx;                                 // per item: exclusive rank among LIST_COPY items
  const u32 *freelist; u32 n_free;           // lowest free destination slots
  u32 *pair_src, *pair_dst;                  // mover pairs, indexed by lidx
  u32 allow_inflight; u32 drop_dead; u32 drop_all;
  u32 reject_shadow;                         // reload: a host slot that is only a copy is not a resident block
  u32 clean_ok;                              // offload: a block with a clean host copy is handed over without a copy
  u32 keep_copy;                             // reload with inclusive tiers: the host slot stays as a clean copy
  u32 w_cut, w_nlive, w_ndrop, w_nclean, w_nshdrop;   // status words this list counts in
  u32 *status;
};
enum : u32 { LIST_DROP = 0, LIST_COPY = 1, LIST_CLEAN = 2 };

__global__ void k_list_validate(ListArgs a) {
  u32 i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= a.n) return;
  u32 id = a.ids[i];
  a.live[i] = LIST_DROP;
  if (id >= a.n_slots) { set_err(a.status, DERR_RANGE); return; }
  u32 e = a.e0 + id;
  if (!a.ent.key[e] || atomicAdd(&a.ent.mark[e], 1u) != 0 || (a.reject_shadow && is_shadow(a.ent, e))) {
    set_err(a.status, DERR_INVAL);
    return;
  }
  if (a.ent.infl[e] && !a.allow_inflight) set_err(a.status, DERR_STATE);
  u32 cat = LIST_COPY;
  if (a.drop_all || (a.drop_dead && entry_rank(a.ent, e) == 0)) cat = LIST_DROP;
  else if (a.clean_ok && a.ent.link[e] != ENT_NONE) cat = LIST_CLEAN;
  a.live[i] = cat;
}

__global__ void k_list_unmark(ListArgs a) {
  u32 i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= a.n) return;
  u32 id = a.ids[i];
  if (id < a.n_slots) a.ent.mark[a.e0 + id] = 0;
}

struct PredLive { const u32 *live; __device__ bool operator()(u32 i) const { return live[i] == LIST_COPY; } };
// item with rank r needs the r-th free destination slot; the first one that does not fit cuts the list
struct EmitLive {
  u32 *lidx; u32 n_free; u32 *cut;
  const u32 *n_free_dev;   // optional: the free count is a device word (computed earlier in the same call)
  __device__ void operator()(u32 i, u32 r) const {
    lidx[i] = r;
    if (r >= (n_free_dev ? min(n_free, *n_free_dev) : n_free)) atomicMin(cut, i);
  }
};
struct PredFree { const u64 *key; u32 e0; __device__ bool operator()(u32 i) const { return key[e0 + i] == 0; } };
struct EmitFree { u32 *list; u32 cap; __device__ void operator()(u32 i, u32 r) const { if (r < cap) list[r] = i; } };

__device__ __forceinline__ void entry_clear(const Entries &en, u32 e) {
  en.key[e] = 0; en.stamp[e] = 0; en.depth[e] = 0; en.infl[e] = 0; en.cnt[e] = 0; en.floor[e] = 0; en.tslot[e] = ENT_NONE;
  en.link[e] = ENT_NONE;
}

// Moves an entry (and whatever points at it: its table slot, its linked copy / block) to a free entry.
__device__ __forceinline__ void entry_move(const Table &t, const Entries &en, u32 src, u32 dst) {
  en.key[dst] = en.key[src]; en.stamp[dst] = en.stamp[src]; en.depth[dst] = en.depth[src];
  en.infl[dst] = en.infl[src]; en.cnt[dst] = en.cnt[src]; en.floor[dst] = en.floor[src];
  u32 s = en.tslot[src];
  en.tslot[dst] = s;
  if (s != ENT_NONE) t.slots[s].ent = dst;
  u32 l = en.link[src];
  en.link[dst] = l;
  if (l != ENT_NONE) en.link[l] = dst;
  entry_clear(en, src);
}

__global__ void k_list_apply(ListArgs a) {
  u32 i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= a.n) return;
  if (a.status[ST_ERR]) return;
  if (i >= a.status[a.w_cut]) return;
  u32 id = a.ids[i];
  u32 e = a.e0 + id;
  u32 cat = a.live[i];
  if (cat == LIST_DROP) {
    if (is_shadow(a.ent, e)) {           // dropping a copy: the block lives on in HBM
      a.ent.link[a.ent.link[e]] = ENT_NONE;
    } else {                             // reclaim without copy: tombstone the key; a clean copy goes too
      u32 s = a.ent.tslot[e];
      a.tab.slots[s].key = KEY_TOMB;
      a.tab.slots[s].ent = ENT_NONE;
      atomicAdd(&a.status[ST_TOMBS], 1u);
      u32 l = a.ent.link[e];
      if (l != ENT_NONE) { entry_clear(a.ent, l); atomicAdd(&a.status[a.w_nshdrop], 1u); }
    }
    entry_clear(a.ent, e);
    atomicAdd(&a.status[a.w_ndrop], 1u);
  } else if (cat == LIST_CLEAN) {        // hand the block over to its clean host copy: metadata only
    u32 h = a.ent.link[e];
    a.ent.stamp[h] = a.ent.stamp[e]; a.ent.depth[h] = a.ent.depth[e]; a.ent.infl[h] = a.ent.infl[e];
    a.ent.cnt[h] = a.ent.cnt[e]; a.ent.floor[h] = a.ent.floor[e];
    u32 s = a.ent.tslot[e];
    a.ent.tslot[h] = s;
    a.tab.slots[s].ent = h;
    a.ent.link[h] = ENT_NONE;
    entry_clear(a.ent, e);
    atomicAdd(&a.status[a.w_nclean], 1u);
  } else {
    u32 r = a.lidx[i];
    KVT_CHECK(r < a.n_free, a.status, return);
    u32 d = a.freelist[r];
    KVT_CHECK(a.ent.key[a.dst_e0 + d] == 0 && a.dst_e0 + d < a.ent.n_total, a.status, return);
    a.pair_src[r] = id;
    a.pair_dst[r] = d;
    u32 de = a.dst_e0 + d;
    if (a.keep_copy) {                   // the block moves to HBM, the host slot stays behind as its clean copy
      a.ent.key[de] = a.ent.key[e]; a.ent.stamp[de] = a.ent.stamp[e]; a.ent.depth[de] = a.ent.depth[e];
      a.ent.infl[de] = a.ent.infl[e]; a.ent.cnt[de] = a.ent.cnt[e]; a.ent.floor[de] = a.ent.floor[e];
      u32 s = a.ent.tslot[e];
      a.ent.tslot[de] = s;
      a.tab.slots[s].ent = de;
      a.ent.link[de] = e;
      a.ent.link[e] = de; a.ent.tslot[e] = ENT_NONE; a.ent.infl[e] = 0; a.ent.cnt[e] = 0;   // a copy carries no state of its own
    } else {
      entry_move(a.tab, a.ent, e, de);
    }
    atomicAdd(&a.status[a.w_nlive], 1u);
  }
}

// ---- compaction plan: i-th occupied slot >= n_occ moves to the i-th free slot < n_occ ---------------
struct PredHole { const u64 *key; u32 e0, n_occ; __device__ bool operator()(u32 i) const { return i < n_occ && key[e0 + i] == 0; } };
struct PredMover { const u64 *key; u32 e0, n_occ; __device__ bool operator()(u32 i) const { return i >= n_occ && key[e0 + i] != 0; } };
struct EmitList { u32 *list; __device__ void operator()(u32 i, u32 r) const { list[r] = i; } };

__global__ void k_compact_apply(Table t, Entries en, u32 e0, const u32 *src, const u32 *dst, const u32 *status) {
  u32 i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= status[ST_NMOVED] || status[ST_ERR]) return;
  KVT_CHECK(e0 + src[i] < en.n_total && e0 + dst[i] < en.n_total && en.key[e0 + src[i]] != 0 && en.key[e0 + dst[i]] == 0,
            const_cast<u32 *>(status), return);
  entry_move(t, en, e0 + src[i], e0 + dst[i]);
}

// ---- debug loader ---------------------------------------------------------------------------------------
struct LoadArgs {
  Table tab; Entries ent; const u64 *keys; const u8 *state; const u32 *stamp, *depth, *slot;
  u32 n, e0, n_slots; u32 *status;
};
__global__ void k_load_check(LoadArgs a) {
  u32 i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= a.n) return;
  if (a.slot[i] >= a.n_slots) { set_err(a.status, DERR_RANGE); return; }
  if (a.ent.key[a.e0 + a.slot[i]]) set_err(a.status, DERR_INVAL);
  if (tab_find(a.tab, a.keys[i], a.status) != ENT_NONE) set_err(a.status, DERR_INVAL);
}
__global__ void k_load_apply(LoadArgs a) {
  u32 i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= a.n || a.status[ST_ERR]) return;
  u32 e = a.e0 + a.slot[i];
  u32 s = tab_find_or_claim(a.tab, a.keys[i], a.status);
  if (s == ENT_NONE) return;
  a.tab.slots[s].ent = e;
  a.ent.key[e] = a.keys[i]; a.ent.stamp[e] = a.stamp[i]; a.ent.depth[e] = a.depth[i];
  a.ent.infl[e] = 0; a.ent.cnt[e] = 0; a.ent.floor[e] = a.state[i]; a.ent.tslot[e] = s; a.ent.link[e] = ENT_NONE;
}

__global__ void k_states_out(Entries en, u32 e0, u32 n, u8 *out) {
  u32 i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = en.key[e0 + i] ? (is_shadow(en, e0 + i) ? (u8)0xFE : (u8)entry_rank(en, e0 + i)) : (u8)0xFF;
}

// ======================================================================================================
// K5: paged KV mover. A pool is addressed as base + slot * slot_stride + chunk * chunk_stride, so the
// layer-major HBM layout, the block-major layout and the host tier all go through the same kernel.
// Work item = (pair, chunk); each CTA streams whole chunks with 16-byte accesses, several loads in
// flight per thread before the first store. The pair count may live in device memory.
// ======================================================================================================
struct PoolView { u8 *base; u64 slot_stride; u64 chunk_stride; u32 n_slots; };
struct MoveArgs {
  PoolView src, dst; const u32 *src_ids, *dst_ids;
  u32 n_pairs; const u32 *n_pairs_dev;   // n_pairs_dev != nullptr: min(*n_pairs_dev, n_pairs)
  u32 n_chunks; u32 chunk_bytes; u32 *status;
};

template <int UNROLL>
__global__ void __launch_bounds__(256) k_move_blocks(MoveArgs a) {
  u32 n_pairs = a.n_pairs;
  if (a.n_pairs_dev) n_pairs = min(n_pairs, *a.n_pairs_dev);
  const u64 n_items = (u64)n_pairs * a.n_chunks;
  const u32 vec_per_chunk = a.chunk_bytes >> 4;
  for (u64 item = blockIdx.x; item < n_items; item += gridDim.x) {
    u32 pair = (u32)(item / a.n_chunks), chunk = (u32)(item % a.n_chunks);
    u32 s = a.src_ids ? a.src_ids[pair] : pair, d = a.dst_ids ? a.dst_ids[pair] : pair;   // no list: the pair's own index
    if (s >= a.src.n_slots || d >= a.dst.n_slots) { if (threadIdx.x == 0) set_err(a.status, DERR_RANGE); continue; }
    const uint4 *sp = reinterpret_cast<const uint4 *>(a.src.base + s * a.src.slot_stride + chunk * a.src.chunk_stride);
    uint4 *dp = reinterpret_cast<uint4 *>(a.dst.base + d * a.dst.slot_stride + chunk * a.dst.chunk_stride);
    for (u32 v0 = threadIdx.x; v0 < vec_per_chunk; v0 += 256 * UNROLL) {
      uint4 r[UNROLL];
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        u32 v = v0 + u * 256;
        if (v < vec_per_chunk) r[u] = __ldcs(sp + v);
      }
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        u32 v = v0 + u * 256;
        if (v < vec_per_chunk) __stcs(dp + v, r[u]);
      }
    }
  }
}

// Variant for small chunks: work item = 32 lanes x 16 B x UNROLL bytes of one chunk, one item per warp
// at a time, so that a 4 KiB chunk keeps UNROLL loads per lane in flight instead of one.
template <int UNROLL, int THREADS = 256>
__global__ void __launch_bounds__(THREADS) k_move_tiles(MoveArgs a, u32 tiles_per_chunk) {
  constexpr u32 WPC = THREADS / 32;   // warps per CTA
  u32 n_pairs = a.n_pairs;
  if (a.n_pairs_dev) n_pairs = min(n_pairs, *a.n_pairs_dev);
  const u32 lane = threadIdx.x & 31;
  const u64 per_pair = (u64)a.n_chunks * tiles_per_chunk;
  const u64 n_items = (u64)n_pairs * per_pair;
  const u64 n_warps = (u64)gridDim.x * WPC;
  for (u64 item = (u64)blockIdx.x * WPC + (threadIdx.x >> 5); item < n_items; item += n_warps) {
    u32 pair = (u32)(item / per_pair);
    u32 rem = (u32)(item - (u64)pair * per_pair);
    u32 chunk = rem / tiles_per_chunk, tile = rem - chunk * tiles_per_chunk;
    u32 s = a.src_ids ? a.src_ids[pair] : pair, d = a.dst_ids ? a.dst_ids[pair] : pair;   // no list: the pair's own index
    if (s >= a.src.n_slots || d >= a.dst.n_slots) { if (lane == 0) set_err(a.status, DERR_RANGE); continue; }
    const uint4 *sp = reinterpret_cast<const uint4 *>(a.src.base + s * a.src.slot_stride + chunk * a.src.chunk_stride) +
                      (u64)tile * 32 * UNROLL + lane;
    uint4 *dp = reinterpret_cast<uint4 *>(a.dst.base + d * a.dst.slot_stride + chunk * a.dst.chunk_stride) +
                (u64)tile * 32 * UNROLL + lane;
    uint4 r[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) r[u] = __ldcs(sp + u * 32);
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) __stcs(dp + u * 32, r[u]);
  }
}

// ---- kvt_exchange: victims out and reloads in with one launch -----------------------------------------------------
// A reload may land in the HBM slot a victim of the same call leaves. vic_of[slot] = index of the victim pair that
// reads that slot; dep[r] = the victim pair reload r has to wait for (ENT_NONE: none); taken[v] = 1: victim v is
// copied out by the warp that copies its successor in.
__global__ void k_xchg_mark(const u32 *vic_src, const u32 *n_vic_dev, u32 n_vic_max, u32 *vic_of, u32 *taken) {
  u32 i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= min(n_vic_max, *n_vic_dev)) return;
  vic_of[vic_src[i]] = i;
  taken[i] = 0;
}
__global__ void k_xchg_link(const u32 *in_dst, const u32 *n_in_dev, u32 n_in_max, const u32 *vic_of, u32 *dep, u32 *taken) {
  u32 r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= min(n_in_max, *n_in_dev)) return;
  u32 v = vic_of[in_dst[r]];
  dep[r] = v;
  if (v != ENT_NONE) taken[v] = 1;
}

// Mover of an exchange. Work unit = one chunk of one pair; two queues (reloads a: host -> HBM, victims b: HBM ->
// host), every warp takes units from both in turn, so both directions of the link are busy whatever the mix. A
// reload unit whose destination slot is being vacated copies that victim's tile out first and then its own tile
// in: the same lane reads and writes the same 16 bytes, so program order keeps the two apart. Victims handled that
// way are skipped in the victim queue.
template <int UNROLL, int THREADS>
__global__ void __launch_bounds__(THREADS) k_move_exchange(MoveArgs a, MoveArgs b, u32 tiles_per_chunk, const u32 *dep,
                                                           const u32 *taken, u32 *queues) {
  u32 na = a.n_pairs, nb = b.n_pairs;
  if (a.n_pairs_dev) na = min(na, *a.n_pairs_dev);
  if (b.n_pairs_dev) nb = min(nb, *b.n_pairs_dev);
  const u32 lane = threadIdx.x & 31;
  const u32 units_a = na * a.n_chunks, units_b = nb * b.n_chunks;
  bool more_a = units_a != 0, more_b = units_b != 0;
  while (more_a || more_b) {
    if (more_a) {
      u32 u = 0;
      if (lane == 0) u = atomicAdd(&queues[0], 1u);
      u = __shfl_sync(0xFFFFFFFFu, u, 0);
      if (u >= units_a) more_a = false;
      else {
        const u32 r = u / a.n_chunks, chunk = u - r * a.n_chunks;
        const u32 v = dep[r];
        const u32 s = a.src_ids[r], d = a.dst_ids[r];
        u32 vs = 0, vd = 0;
        bool ok = s < a.src.n_slots && d < a.dst.n_slots;
        if (v != ENT_NONE) { vs = b.src_ids[v]; vd = b.dst_ids[v]; ok = ok && vs < b.src.n_slots && vd < b.dst.n_slots; }
        if (!ok) { if (lane == 0) set_err(a.status, DERR_RANGE); }
        else {
          const uint4 *sp = reinterpret_cast<const uint4 *>(a.src.base + s * a.src.slot_stride + chunk * a.src.chunk_stride) + lane;
          uint4 *dp = reinterpret_cast<uint4 *>(a.dst.base + d * a.dst.slot_stride + chunk * a.dst.chunk_stride) + lane;
          const uint4 *vsp = reinterpret_cast<const uint4 *>(b.src.base + vs * b.src.slot_stride + chunk * b.src.chunk_stride) + lane;
          uint4 *vdp = reinterpret_cast<uint4 *>(b.dst.base + vd * b.dst.slot_stride + chunk * b.dst.chunk_stride) + lane;
          for (u32 t = 0; t < tiles_per_chunk; ++t) {
            const u64 o = (u64)t * 32 * UNROLL;
            uint4 x[UNROLL];
            if (v != ENT_NONE) {        // the victim's tile leaves before the new one overwrites it
#pragma unroll
              for (int q = 0; q < UNROLL; ++q) x[q] = __ldcs(vsp + o + q * 32);
#pragma unroll
              for (int q = 0; q < UNROLL; ++q) __stcs(vdp + o + q * 32, x[q]);
            }
#pragma unroll
            for (int q = 0; q < UNROLL; ++q) x[q] = __ldcs(sp + o + q * 32);
#pragma unroll
            for (int q = 0; q < UNROLL; ++q) __stcs(dp + o + q * 32, x[q]);
          }
        }
      }
    }
    if (more_b) {
      u32 u = 0;
      if (lane == 0) u = atomicAdd(&queues[1], 1u);
      u = __shfl_sync(0xFFFFFFFFu, u, 0);
      if (u >= units_b) more_b = false;
      else {
        const u32 v = u / b.n_chunks, chunk = u - v * b.n_chunks;
        if (!taken[v]) {
          const u32 s = b.src_ids[v], d = b.dst_ids[v];
          if (s >= b.src.n_slots || d >= b.dst.n_slots) { if (lane == 0) set_err(b.status, DERR_RANGE); }
          else {
            const uint4 *sp = reinterpret_cast<const uint4 *>(b.src.base + s * b.src.slot_stride + chunk * b.src.chunk_stride) + lane;
            uint4 *dp = reinterpret_cast<uint4 *>(b.dst.base + d * b.dst.slot_stride + chunk * b.dst.chunk_stride) + lane;
            for (u32 t = 0; t < tiles_per_chunk; ++t) {
              const u64 o = (u64)t * 32 * UNROLL;
              uint4 x[UNROLL];
#pragma unroll
              for (int q = 0; q < UNROLL; ++q) x[q] = __ldcs(sp + o + q * 32);
#pragma unroll
              for (int q = 0; q < UNROLL; ++q) __stcs(dp + o + q * 32, x[q]);
            }
          }
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------------
// TMA variant: one elected thread per CTA drives a ring of shared-memory stages with untiled bulk copies
// (cp.async.bulk global -> shared, completion on an mbarrier; shared -> global as a bulk group). No registers
// carry payload; every wait is bounded and reports through the status word. Every copy is CTA-local: one source, one destination, no clusters.
// ------------------------------------------------------------------------------------------------------
constexpr int TMA_STAGES = 4;

__global__ void __launch_bounds__(32) k_move_tma(MoveArgs a, u32 tile_bytes, u32 tiles_per_chunk) {
  extern __shared__ __align__(128) u8 smem[];
  __shared__ __align__(8) u64 bars[TMA_STAGES];
  if (threadIdx.x != 0) return;            // one thread issues everything; the copies run in the async proxy
  u32 n_pairs = a.n_pairs;
  if (a.n_pairs_dev) n_pairs = min(n_pairs, *a.n_pairs_dev);
  const u64 per_pair = (u64)a.n_chunks * tiles_per_chunk;
  const u64 n_items = (u64)n_pairs * per_pair;
  if (blockIdx.x >= n_items) return;
  const u64 n_mine = (n_items - blockIdx.x + gridDim.x - 1) / gridDim.x;   // my tiles: blockIdx + k * gridDim
  for (int s = 0; s < TMA_STAGES; ++s) mbar_init(&bars[s], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");

  auto locate = [&](u64 k, const u8 *&src, u8 *&dst) -> bool {
    u64 item = blockIdx.x + k * gridDim.x;
    u32 pair = (u32)(item / per_pair);
    u32 rem = (u32)(item - (u64)pair * per_pair);
    u32 chunk = rem / tiles_per_chunk, tile = rem - chunk * tiles_per_chunk;
    u32 sid = a.src_ids[pair], did = a.dst_ids[pair];
    if (sid >= a.src.n_slots || did >= a.dst.n_slots) { set_err(a.status, DERR_RANGE); return false; }
    src = a.src.base + sid * a.src.slot_stride + chunk * a.src.chunk_stride + (u64)tile * tile_bytes;
    dst = a.dst.base + did * a.dst.slot_stride + chunk * a.dst.chunk_stride + (u64)tile * tile_bytes;
    return true;
  };
  auto issue_load = [&](u64 k) {
    const u8 *src; u8 *dst;
    int s = (int)(k % TMA_STAGES);
    if (locate(k, src, dst)) {
      mbar_expect_tx(&bars[s], tile_bytes);
      bulk_load(smem + (size_t)s * tile_bytes, src, tile_bytes, &bars[s]);
    } else {
      mbar_expect_tx(&bars[s], 0);          // keep the phase sequence going for a skipped tile
    }
  };

  const u64 prologue = n_mine < TMA_STAGES ? n_mine : TMA_STAGES;
  for (u64 k = 0; k < prologue; ++k) issue_load(k);
  bool ok = true;
  for (u64 k = 0; k < n_mine && ok; ++k) {
    int s = (int)(k % TMA_STAGES);
    ok = mbar_wait(&bars[s], (u32)((k / TMA_STAGES) & 1));
    if (!ok) break;
    const u8 *src; u8 *dst;
    if (locate(k, src, dst)) bulk_store(dst, smem + (size_t)s * tile_bytes, tile_bytes);
    else asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    // the stage of tile k-1 may be refilled once its store has finished reading shared memory
    if (k >= 1 && k - 1 + TMA_STAGES < n_mine) {
      asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      issue_load(k - 1 + TMA_STAGES);
    }
  }
  if (!ok) set_err(a.status, DERR_PROBE);
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all my stores are complete before the CTA ends
}

}  // namespace kvt
