// Host-side caches of the serving loop around the decode step: the text prefix cache (Algorithm 2) over the paged
// KV pool, and the content-hash store of the multimodal path (Algorithm 3), both bounded by an LRU byte budget
// (Section 3.3, "Memory Management": 512 MB by default).
//
// Text prefix cache.  Algorithm 2 hashes the whole prompt, then every shorter prefix, and returns the KV state of the
// longest prefix it finds together with the position to resume from.  Here the KV state of a prefix is a list of
// 16-token blocks of the pool, an entry exists for every block-aligned prefix that was inserted, and the key of the
// prefix ending with block i is SHA-256(key of the prefix ending with block i-1 || the block's 16 token ids): one
// hash per block instead of one per prefix length, the same hits (a prefix is found exactly when all of its blocks
// are), and prompts that share a prefix share its blocks.  Blocks belong to the caller's pool: the cache hands out
// block ids, counts who is reading them, and names the blocks it gives up when it evicts.
#include <stdint.h>
#include <string.h>

#include <new>
#include <unordered_map>
#include <vector>

#include "../../include/q4decode.h"

extern "C" int q4d_internal_fail(int code, const char* msg);

namespace {

// ---- SHA-256 (FIPS 180-4) ------------------------------------------------------------
struct Sha256 {
  uint32_t h[8];
  uint8_t buf[64];
  uint64_t total;
  size_t fill;
};
const uint32_t kRound[64] = {
    0x428a2f98, 0x71374491, 0xb5c0fbcf, 0xe9b5dba5, 0x3956c25b, 0x59f111f1, 0x923f82a4, 0xab1c5ed5, 0xd807aa98, 0x12835b01,
    0x243185be, 0x550c7dc3, 0x72be5d74, 0x80deb1fe, 0x9bdc06a7, 0xc19bf174, 0xe49b69c1, 0xefbe4786, 0x0fc19dc6, 0x240ca1cc,
    0x2de92c6f, 0x4a7484aa, 0x5cb0a9dc, 0x76f988da, 0x983e5152, 0xa831c66d, 0xb00327c8, 0xbf597fc7, 0xc6e00bf3, 0xd5a79147,
    0x06ca6351, 0x14292967, 0x27b70a85, 0x2e1b2138, 0x4d2c6dfc, 0x53380d13, 0x650a7354, 0x766a0abb, 0x81c2c92e, 0x92722c85,
    0xa2bfe8a1, 0xa81a664b, 0xc24b8b70, 0xc76c51a3, 0xd192e819, 0xd6990624, 0xf40e3585, 0x106aa070, 0x19a4c116, 0x1e376c08,
    0x2748774c, 0x34b0bcb5, 0x391c0cb3, 0x4ed8aa4a, 0x5b9cca4f, 0x682e6ff3, 0x748f82ee, 0x78a5636f, 0x84c87814, 0x8cc70208,
    0x90befffa, 0xa4506ceb, 0xbef9a3f7, 0xc67178f2};
inline uint32_t rotr(uint32_t x, int n) { return (x >> n) | (x << (32 - n)); }

void sha_block(Sha256& s, const uint8_t* p) {
  uint32_t w[64];
  for (int i = 0; i < 16; ++i) w[i] = (uint32_t)p[4 * i] << 24 | (uint32_t)p[4 * i + 1] << 16 | (uint32_t)p[4 * i + 2] << 8 | p[4 * i + 3];
  for (int i = 16; i < 64; ++i) {
    const uint32_t s0 = rotr(w[i - 15], 7) ^ rotr(w[i - 15], 18) ^ (w[i - 15] >> 3);
    const uint32_t s1 = rotr(w[i - 2], 17) ^ rotr(w[i - 2], 19) ^ (w[i - 2] >> 10);
    w[i] = w[i - 16] + s0 + w[i - 7] + s1;
  }
  uint32_t a = s.h[0], b = s.h[1], c = s.h[2], d = s.h[3], e = s.h[4], f = s.h[5], g = s.h[6], hh = s.h[7];
  for (int i = 0; i < 64; ++i) {
    const uint32_t t1 = hh + (rotr(e, 6) ^ rotr(e, 11) ^ rotr(e, 25)) + ((e & f) ^ (~e & g)) + kRound[i] + w[i];
    const uint32_t t2 = (rotr(a, 2) ^ rotr(a, 13) ^ rotr(a, 22)) + ((a & b) ^ (a & c) ^ (b & c));
    hh = g, g = f, f = e, e = d + t1, d = c, c = b, b = a, a = t1 + t2;
  }
  s.h[0] += a, s.h[1] += b, s.h[2] += c, s.h[3] += d, s.h[4] += e, s.h[5] += f, s.h[6] += g, s.h[7] += hh;
}
void sha_init(Sha256& s) {
  const uint32_t iv[8] = {0x6a09e667, 0xbb67ae85, 0x3c6ef372, 0xa54ff53a, 0x510e527f, 0x9b05688c, 0x1f83d9ab, 0x5be0cd19};
  memcpy(s.h, iv, sizeof iv);
  s.total = 0, s.fill = 0;
}
void sha_update(Sha256& s, const void* data, size_t n) {
  const uint8_t* p = static_cast<const uint8_t*>(data);
  s.total += n;
  while (n) {
    const size_t take = n < 64 - s.fill ? n : 64 - s.fill;
    memcpy(s.buf + s.fill, p, take);
    s.fill += take, p += take, n -= take;
    if (s.fill == 64) sha_block(s, s.buf), s.fill = 0;
  }
}
void sha_final(Sha256& s, uint8_t out[32]) {
  const uint64_t bits = s.total * 8;
  const uint8_t one = 0x80, zero = 0;
  sha_update(s, &one, 1);
  while (s.fill != 56) sha_update(s, &zero, 1);
  uint8_t len[8];
  for (int i = 0; i < 8; ++i) len[i] = (uint8_t)(bits >> (56 - 8 * i));
  sha_update(s, len, 8);
  for (int i = 0; i < 8; ++i)
    out[4 * i] = (uint8_t)(s.h[i] >> 24), out[4 * i + 1] = (uint8_t)(s.h[i] >> 16), out[4 * i + 2] = (uint8_t)(s.h[i] >> 8),
             out[4 * i + 3] = (uint8_t)s.h[i];
}

struct Digest {
  uint8_t b[32];
  bool operator==(const Digest& o) const { return memcmp(b, o.b, 32) == 0; }
};
struct DigestHash {
  size_t operator()(const Digest& d) const {
    size_t v;
    memcpy(&v, d.b, sizeof v);
    return v;
  }
};

constexpr size_t kDefaultCapacity = 512ull << 20;  // Section 3.3: 512 MB unless configured

}  // namespace

// ---- text prefix cache -----------------------------------------------------------------

struct q4d_prefix_cache {
  struct Entry {
    Digest key;
    int32_t block, parent, children, readers;
    uint64_t last_use;
    bool live;
  };
  size_t capacity, bytes_per_block;
  std::vector<Entry> entries;
  std::vector<int32_t> free_slots;
  std::unordered_map<Digest, int32_t, DigestHash> index;
  uint64_t clock = 0;
  int64_t live = 0, lookups = 0, hit_blocks = 0;

  static Digest chain(const Digest* parent, const int32_t* block_tokens) {
    Sha256 s;
    sha_init(s);
    if (parent) sha_update(s, parent->b, 32);
    sha_update(s, block_tokens, Q4D_BLOCK_SIZE * sizeof(int32_t));
    Digest d;
    sha_final(s, d.b);
    return d;
  }
};

extern "C" {

int q4d_sha256(const void* data, size_t bytes, uint8_t* out32) {
  if ((!data && bytes) || !out32) return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "sha256: NULL argument");
  Sha256 s;
  sha_init(s);
  sha_update(s, data, bytes);
  sha_final(s, out32);
  return Q4D_OK;
}

int q4d_prefix_cache_create(size_t capacity_bytes, size_t bytes_per_block, q4d_prefix_cache** out) {
  if (!out || bytes_per_block == 0) return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "prefix_cache_create: bad argument");
  q4d_prefix_cache* c = new (std::nothrow) q4d_prefix_cache();
  if (!c) return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "prefix_cache_create: out of host memory");
  c->capacity = capacity_bytes ? capacity_bytes : kDefaultCapacity;
  c->bytes_per_block = bytes_per_block;
  *out = c;
  return Q4D_OK;
}

int q4d_prefix_cache_destroy(q4d_prefix_cache* c) {
  delete c;
  return Q4D_OK;
}

int q4d_prefix_lookup(q4d_prefix_cache* c, const int32_t* tokens, int32_t n_tokens, int32_t max_blocks, int32_t* blocks_out,
                      int32_t* handles_out, int32_t* n_hit_blocks) {
  if (!c || (!tokens && n_tokens) || n_tokens < 0 || max_blocks < 0 || !n_hit_blocks || (max_blocks && (!blocks_out || !handles_out)))
    return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "prefix_lookup: bad argument");
  c->lookups++;
  const int32_t full = n_tokens / Q4D_BLOCK_SIZE;
  int32_t hit = 0;
  Digest prev;
  for (int32_t i = 0; i < full && i < max_blocks; ++i) {
    const Digest key = q4d_prefix_cache::chain(i ? &prev : nullptr, tokens + (size_t)i * Q4D_BLOCK_SIZE);
    auto it = c->index.find(key);
    if (it == c->index.end()) break;
    q4d_prefix_cache::Entry& e = c->entries[it->second];
    e.readers++;
    e.last_use = ++c->clock;
    blocks_out[i] = e.block, handles_out[i] = it->second;
    prev = key;
    hit = i + 1;
  }
  c->hit_blocks += hit;
  *n_hit_blocks = hit;
  return Q4D_OK;
}

int q4d_prefix_insert(q4d_prefix_cache* c, const int32_t* tokens, int32_t n_tokens, const int32_t* block_table,
                      int32_t n_blocks, int32_t* handles_out, int32_t* adopted_out) {
  if (!c || !tokens || n_tokens < 0 || !block_table || n_blocks < 0 || !handles_out || !adopted_out)
    return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "prefix_insert: bad argument");
  const int32_t full = n_tokens / Q4D_BLOCK_SIZE;
  if (n_blocks > full) n_blocks = full;
  Digest prev;
  int32_t parent = -1;
  for (int32_t i = 0; i < n_blocks; ++i) {
    const Digest key = q4d_prefix_cache::chain(i ? &prev : nullptr, tokens + (size_t)i * Q4D_BLOCK_SIZE);
    prev = key;
    auto it = c->index.find(key);
    if (it != c->index.end()) {
      // this prefix is cached already (by a block of someone else, or by this very block after a lookup)
      q4d_prefix_cache::Entry& e = c->entries[it->second];
      handles_out[i] = -1, adopted_out[i] = e.block == block_table[i] ? 1 : 0;
      e.last_use = ++c->clock;
      parent = it->second;
      continue;
    }
    int32_t slot;
    if (!c->free_slots.empty()) {
      slot = c->free_slots.back();
      c->free_slots.pop_back();
    } else {
      slot = (int32_t)c->entries.size();
      c->entries.emplace_back();
    }
    q4d_prefix_cache::Entry& e = c->entries[slot];
    e.key = key, e.block = block_table[i], e.parent = parent, e.children = 0, e.readers = 1, e.live = true;
    e.last_use = ++c->clock;
    if (parent >= 0) c->entries[parent].children++;
    c->index.emplace(key, slot);
    c->live++;
    handles_out[i] = slot, adopted_out[i] = 1;
    parent = slot;
  }
  return Q4D_OK;
}

int q4d_prefix_release(q4d_prefix_cache* c, const int32_t* handles, int32_t n) {
  if (!c || (!handles && n) || n < 0) return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "prefix_release: bad argument");
  for (int32_t i = 0; i < n; ++i) {
    const int32_t h = handles[i];
    if (h < 0) continue;
    if (h >= (int32_t)c->entries.size() || !c->entries[h].live || c->entries[h].readers < 1)
      return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "prefix_release: handle is not held");
    c->entries[h].readers--;
  }
  return Q4D_OK;
}

int q4d_prefix_evict(q4d_prefix_cache* c, size_t bytes_to_free, int32_t max_out, int32_t* freed_blocks, int32_t* n_freed) {
  if (!c || max_out < 0 || (max_out && !freed_blocks) || !n_freed)
    return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "prefix_evict: bad argument");
  const size_t held = (size_t)c->live * c->bytes_per_block;
  // down to the capacity, or by the requested amount if that is more
  size_t target = held > c->capacity ? held - c->capacity : 0;
  if (bytes_to_free > target) target = bytes_to_free;
  int32_t out = 0;
  size_t freed = 0;
  while (freed < target && out < max_out) {
    // least recently used entry that nobody reads and that no longer prefix depends on
    int32_t victim = -1;
    for (int32_t i = 0; i < (int32_t)c->entries.size(); ++i) {
      const q4d_prefix_cache::Entry& e = c->entries[i];
      if (e.live && e.readers == 0 && e.children == 0 && (victim < 0 || e.last_use < c->entries[victim].last_use)) victim = i;
    }
    if (victim < 0) break;
    q4d_prefix_cache::Entry& e = c->entries[victim];
    if (e.parent >= 0) c->entries[e.parent].children--;
    c->index.erase(e.key);
    e.live = false;
    c->free_slots.push_back(victim);
    c->live--;
    freed_blocks[out++] = e.block;
    freed += c->bytes_per_block;
  }
  *n_freed = out;
  return Q4D_OK;
}

int q4d_prefix_cache_stats(q4d_prefix_cache* c, int64_t* entries, int64_t* bytes, int64_t* lookups, int64_t* hit_blocks) {
  if (!c) return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "prefix_cache_stats: NULL cache");
  if (entries) *entries = c->live;
  if (bytes) *bytes = c->live * (int64_t)c->bytes_per_block;
  if (lookups) *lookups = c->lookups;
  if (hit_blocks) *hit_blocks = c->hit_blocks;
  return Q4D_OK;
}

}  // extern "C"

// ---- content-hash store of the multimodal path ------------------------------------------

struct q4d_content_cache {
  struct Entry {
    q4d_content_entry payload;
    std::vector<int32_t> blocks;
    int32_t readers;
    uint64_t last_use;
  };
  size_t capacity, bytes = 0;
  std::unordered_map<Digest, Entry, DigestHash> map;
  uint64_t clock = 0;
};

extern "C" {

int q4d_content_cache_create(size_t capacity_bytes, q4d_content_cache** out) {
  if (!out) return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "content_cache_create: NULL argument");
  q4d_content_cache* c = new (std::nothrow) q4d_content_cache();
  if (!c) return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "content_cache_create: out of host memory");
  c->capacity = capacity_bytes ? capacity_bytes : kDefaultCapacity;
  *out = c;
  return Q4D_OK;
}

int q4d_content_cache_destroy(q4d_content_cache* c) {
  delete c;
  return Q4D_OK;
}

int q4d_content_lookup(q4d_content_cache* c, const void* pixels, size_t pixel_bytes, q4d_content_entry* entry_out,
                       int32_t max_blocks, int32_t* blocks_out, int32_t* hit) {
  if (!c || !pixels || !entry_out || !hit || max_blocks < 0 || (max_blocks && !blocks_out))
    return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "content_lookup: bad argument");
  Digest key;
  q4d_sha256(pixels, pixel_bytes, key.b);
  memcpy(entry_out->hash, key.b, 32);
  auto it = c->map.find(key);
  if (it == c->map.end()) {
    *hit = 0;
    return Q4D_OK;
  }
  q4d_content_cache::Entry& e = it->second;
  if ((int32_t)e.blocks.size() > max_blocks) return q4d_internal_fail(Q4D_ERR_BLOCK_TABLE_TOO_SHORT, "content_lookup: blocks_out too short");
  e.readers++;
  e.last_use = ++c->clock;
  *entry_out = e.payload;
  for (size_t i = 0; i < e.blocks.size(); ++i) blocks_out[i] = e.blocks[i];
  *hit = 1;
  return Q4D_OK;
}

int q4d_content_store(q4d_content_cache* c, const q4d_content_entry* entry, const int32_t* blocks) {
  if (!c || !entry || entry->n_blocks < 0 || (entry->n_blocks && !blocks))
    return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "content_store: bad argument");
  Digest key;
  memcpy(key.b, entry->hash, 32);
  if (c->map.count(key)) return q4d_internal_fail(Q4D_ERR_DUPLICATE_REQUEST, "content_store: this content is cached already");
  q4d_content_cache::Entry e;
  e.payload = *entry;
  e.blocks.assign(blocks, blocks + entry->n_blocks);
  e.readers = 1;  // the storing request is still using it
  e.last_use = ++c->clock;
  c->bytes += (size_t)entry->bytes;
  c->map.emplace(key, std::move(e));
  return Q4D_OK;
}

int q4d_content_release(q4d_content_cache* c, const uint8_t* hash32) {
  if (!c || !hash32) return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "content_release: NULL argument");
  Digest key;
  memcpy(key.b, hash32, 32);
  auto it = c->map.find(key);
  if (it == c->map.end() || it->second.readers < 1) return q4d_internal_fail(Q4D_ERR_UNKNOWN_REQUEST, "content_release: entry is not held");
  it->second.readers--;
  return Q4D_OK;
}

int q4d_content_evict(q4d_content_cache* c, size_t bytes_to_free, q4d_content_entry* evicted_out, int32_t max_blocks,
                      int32_t* blocks_out, int32_t* did_evict) {
  if (!c || !evicted_out || !did_evict || max_blocks < 0 || (max_blocks && !blocks_out))
    return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "content_evict: bad argument");
  *did_evict = 0;
  if (c->bytes <= c->capacity && bytes_to_free == 0) return Q4D_OK;
  auto victim = c->map.end();
  for (auto it = c->map.begin(); it != c->map.end(); ++it)
    if (it->second.readers == 0 && (victim == c->map.end() || it->second.last_use < victim->second.last_use)) victim = it;
  if (victim == c->map.end()) return Q4D_OK;
  if ((int32_t)victim->second.blocks.size() > max_blocks) return q4d_internal_fail(Q4D_ERR_BLOCK_TABLE_TOO_SHORT, "content_evict: blocks_out too short");
  *evicted_out = victim->second.payload;
  for (size_t i = 0; i < victim->second.blocks.size(); ++i) blocks_out[i] = victim->second.blocks[i];
  c->bytes -= (size_t)victim->second.payload.bytes;
  c->map.erase(victim);
  *did_evict = 1;
  return Q4D_OK;
}

int q4d_content_cache_stats(q4d_content_cache* c, int64_t* entries, int64_t* bytes) {
  if (!c) return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "content_cache_stats: NULL cache");
  if (entries) *entries = (int64_t)c->map.size();
  if (bytes) *bytes = (int64_t)c->bytes;
  return Q4D_OK;
}

}  // extern "C"
