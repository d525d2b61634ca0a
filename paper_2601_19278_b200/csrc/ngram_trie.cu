// The N-gram as child lists in device memory (Appendix C: a trie whose context node is located once and whose
// children are then read for all candidates).  Host side: sort the rows by (order, a, b, t), drop repeated rows
// (the first stays), and write the lists back to back -- a compressed-sparse-row trie:
//   * 2-gram rows (b, t):    offsets by b, entries {t, score};
//   * 3-gram rows (a, b, t): offsets by a into the context nodes {b, first child}, entries {t, score}.
// 8 bytes per row and 8 per distinct 3-gram context, against 32 bytes per row of the hash table at load 0.5.
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

cudaError_t ngram_trie_build(const unsigned char* order, const int32_t* c0, const int32_t* c1, const int32_t* nx, const float* score,
                             long long n_rows, int vocab, int ngram_order, NgramTrieOwned* out) {
  *out = NgramTrieOwned{};
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
  unsigned long long last = 0ull;   // no row has key 0
  int last_a = -1, last_b = -1;
  for (const auto& kr : rows) {
    if (kr.first == last) continue;
    last = kr.first;
    const uint32_t i = kr.second;
    uint32_t sbits;
    memcpy(&sbits, &score[i], 4);
    if (order[i] == 2) {
      bi_ent.push_back(make_uint2((uint32_t)nx[i], sbits));
      bi_off[(size_t)c1[i] + 1] += 1;
    } else {
      if (c0[i] != last_a || c1[i] != last_b) {
        last_a = c0[i]; last_b = c1[i];
        tri_node.push_back(make_uint2((uint32_t)c1[i], (uint32_t)tri_ent.size()));
        tri_off[(size_t)c0[i] + 1] += 1;
      }
      tri_ent.push_back(make_uint2((uint32_t)nx[i], sbits));
    }
  }
  tri_node.push_back(make_uint2(0x7fffffffu, (uint32_t)tri_ent.size()));   // sentinel: where the last node's children end
  for (int v = 0; v < vocab; ++v) { bi_off[v + 1] += bi_off[v]; tri_off[v + 1] += tri_off[v]; }
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
