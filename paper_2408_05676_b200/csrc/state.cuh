// Internal definitions of the opaque handles shared between translation units.
#pragma once
#include <cuda.h>

#include "common.cuh"

struct laser_kv {
  int32_t n_layers = 0, n_kv_heads = 0, head_dim = 0, page_size = 16;
  int32_t max_seqs = 0, pages_per_seq = 0;
  int64_t n_pages = 0;
  // pages: [layer][page][K|V][kv_head][token-in-page][head_dim] bf16
  __nv_bfloat16* pages = nullptr;
  int32_t* page_table = nullptr;  // dev [max_seqs, pages_per_seq]
  int32_t* seq_len = nullptr;     // dev [max_seqs] committed tokens
  // all pages as one 2-D bf16 matrix [rows of head_dim]: TMA source of the attention kernel
  CUtensorMap pages_map{};
  bool has_pages_map = false;
  size_t page_elems() const { return size_t(2) * n_kv_heads * page_size * head_dim; }
  size_t layer_elems() const { return size_t(n_pages) * page_elems(); }
  int64_t capacity_tokens() const { return int64_t(pages_per_seq) * page_size; }
};
