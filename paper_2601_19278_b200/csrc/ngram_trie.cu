// The N-gram as child lists in device memory (Appendix C: a trie whose context node is located once and whose
// children are then read for all candidates).  Host side: sort the rows by (order, a, b, t), drop repeated rows
// (the first stays), and write the lists back to back -- a compressed-sparse-row trie:
//   * 2-gram rows (b, t):    offsets by b, entries {t, score};
//   * 3-gram rows (a, b, t): offsets by a into the context nodes {b, first child}, entries {t, score}.
// A list of more than kTrieLongList entries is preceded by a bitmap of the tokens it holds, in 64-byte blocks of a
// running count and 480 bits, so that any of its entries is two dependent reads away whatever its length (block,
// then entry); shorter lists are read whole.  8 bytes per row, 8 per distinct 3-gram context and 64 bytes per 480
// vocabulary entries for each long list, against 32 bytes per row of the hash table at load 0.5.
#include <algorithm>
#include <cstring>
#include <utility>
#include <vector>

#include "common.cuh"
#include "kernels.h"

namespace dart {

void ngram_trie_free(NgramTrieOwned* t) {
  if (t == nullptr) return;
  if (t->bi_off) cudaFree(t->bi_off);
  if (t->bi_ent) cudaFree(t->bi_ent);
  if (t->tri_off) cudaFree(t->tri_off);
  if (t->tri_node) cudaFree(t->tri_node);
  if (t->tri_ent) cudaFree(t->tri_ent);
  *t = NgramTrieOwned{};
}

template <typename T>
static cudaError_t upload(T** dst, const std::vector<T>& src, size_t* bytes) {
  const size_t n = src.size() * sizeof(T);
  cudaError_t e = cudaMalloc(dst, n > 0 ? n : sizeof(T));
  if (e != cudaSuccess) return e;
  *bytes += n;
  return n > 0 ? cudaMemcpy(*dst, src.data(), n, cudaMemcpyHostToDevice) : cudaSuccess;
}

namespace {

// Append one list's region to `arr`; returns where the region starts.  A long list's region is aligned to 64 bytes
// (the slots skipped over carry a token no lookup asks for and fall into the previous region) and starts with the
// bitmap blocks (which index the items, not the tail).  `tail`, a sentinel entry, follows the items when with_tail.
uint32_t append_list(std::vector<uint2>& arr, const std::vector<uint2>& items, int n_blocks, bool with_tail, uint2 tail) {
  const size_t n = items.size() + (with_tail ? 1 : 0);
  if (n > (size_t)kTrieLongList) {
    while (arr.size() % 8 != 0) arr.push_back(make_uint2(0xffffffffu, 0u));
    const size_t start = arr.size();
    arr.resize(start + (size_t)n_blocks * 8, make_uint2(0u, 0u));
    uint32_t* words = reinterpret_cast<uint32_t*>(arr.data() + start);   // n_blocks x 16 words
    for (const uint2& it : items) {
      const uint32_t blk = it.x / 480u, r = it.x % 480u;
      words[(size_t)blk * 16 + 1 + (r >> 5)] |= 1u << (r & 31u);
    }
    uint32_t running = 0;
    for (int blk = 0; blk < n_blocks; ++blk) {
      words[(size_t)blk * 16] = running;
      for (int q = 1; q < 16; ++q) running += (uint32_t)__builtin_popcount(words[(size_t)blk * 16 + q]);
    }
    arr.insert(arr.end(), items.begin(), items.end());
    if (with_tail) arr.push_back(tail);
    return (uint32_t)start;
  }
  const size_t start = arr.size();
  arr.insert(arr.end(), items.begin(), items.end());
  if (with_tail) arr.push_back(tail);
  return (uint32_t)start;
}

}  // namespace

cudaError_t ngram_trie_build(const unsigned char* order, const int32_t* c0, const int32_t* c1, const int32_t* nx, const float* score,
                             long long n_rows, int vocab, int ngram_order, NgramTrieOwned* out) {
  *out = NgramTrieOwned{};
  const int n_blocks = (vocab + 479) / 480;
  // (sort key, row): the key orders rows by (order, a, b, t); equal keys keep their row order, so the first stays
  std::vector<std::pair<unsigned long long, uint32_t>> rows;
  rows.reserve((size_t)n_rows);
  for (long long i = 0; i < n_rows; ++i) {
    if (order[i] == 3 && ngram_order < 3) continue;
    rows.emplace_back(ngram_key(order[i], c0[i], c1[i], nx[i]), (uint32_t)i);
  }
  std::sort(rows.begin(), rows.end());

  std::vector<uint32_t> bi_off((size_t)vocab + 1, 0u), tri_off((size_t)vocab + 1, 0u);
  std::vector<uint2> bi_ent, tri_node, tri_ent;
  std::vector<uint2> items, nodes;        // the list being collected: children of one context / nodes of one first token
  // the sorted rows fall into runs: 2-gram rows by b; 3-gram rows by a, inside a run of a by b
  size_t r = 0;
  const size_t R = rows.size();
  auto same_row = [&](size_t x, size_t y) { return rows[x].first == rows[y].first; };
  int next_b = 0, next_a = 0;             // offsets filled up to here
  while (r < R && order[rows[r].second] == 2) {
    const int b = c1[rows[r].second];
    items.clear();
    while (r < R && order[rows[r].second] == 2 && c1[rows[r].second] == b) {
      const uint32_t i = rows[r].second;
      uint32_t sbits;
      memcpy(&sbits, &score[i], 4);
      items.push_back(make_uint2((uint32_t)nx[i], sbits));
      do { ++r; } while (r < R && same_row(r, r - 1));
    }
    const uint32_t start = append_list(bi_ent, items, n_blocks, false, make_uint2(0u, 0u));
    for (; next_b <= b; ++next_b) bi_off[next_b] = start;
  }
  for (; next_b <= vocab; ++next_b) bi_off[next_b] = (uint32_t)bi_ent.size();
  while (r < R) {
    const int a = c0[rows[r].second];
    nodes.clear();
    while (r < R && c0[rows[r].second] == a) {
      const int b = c1[rows[r].second];
      items.clear();
      while (r < R && c0[rows[r].second] == a && c1[rows[r].second] == b) {
        const uint32_t i = rows[r].second;
        uint32_t sbits;
        memcpy(&sbits, &score[i], 4);
        items.push_back(make_uint2((uint32_t)nx[i], sbits));
        do { ++r; } while (r < R && same_row(r, r - 1));
      }
      nodes.push_back(make_uint2((uint32_t)b, append_list(tri_ent, items, n_blocks, false, make_uint2(0u, 0u))));
    }
    // every node's children end where the next node's begin; the list's own sentinel says where the last node's end
    const uint32_t start = append_list(tri_node, nodes, n_blocks, true, make_uint2(0x7fffffffu, (uint32_t)tri_ent.size()));
    for (; next_a <= a; ++next_a) tri_off[next_a] = start;
  }
  for (; next_a <= vocab; ++next_a) tri_off[next_a] = (uint32_t)tri_node.size();
  rows.clear(); rows.shrink_to_fit();

  cudaError_t e;
  size_t bytes = 0;
  if ((e = upload(&out->bi_off, bi_off, &bytes)) != cudaSuccess || (e = upload(&out->bi_ent, bi_ent, &bytes)) != cudaSuccess ||
      (e = upload(&out->tri_off, tri_off, &bytes)) != cudaSuccess || (e = upload(&out->tri_node, tri_node, &bytes)) != cudaSuccess ||
      (e = upload(&out->tri_ent, tri_ent, &bytes)) != cudaSuccess) {
    ngram_trie_free(out);
    return e;
  }
  out->bytes = bytes;
  return cudaSuccess;
}

}  // namespace dart
