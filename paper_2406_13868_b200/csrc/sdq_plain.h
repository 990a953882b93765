// Buffer layout of the decompose-only reading (element-wise 2:4 inliers): the canonical arrays themselves, one code
// per byte.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "sdq_internal.h"
#include "sdq_layout.h"

namespace sdq {

// pair-wise 4:8 inliers with one scale per 64 K (kind::mxf4 .block32) or per 32 K (kind::mxf4nvf4 .block16), or dense
// inliers with one scale per 32 K (dense kind::mxf4 .block32), which also carries element-wise 2:4 inliers with one
// scale per 32 K: tiled layout
inline bool is_tensor_core_reading(const sdq_config_t& c) {
  return (c.in_gran == SDQ_GRAN_PAIR && (c.in_block == 64 || c.in_block == 32)) || (c.in_gran >= SDQ_GRAN_DENSE && c.in_block == 32) ||
         (c.in_gran == SDQ_GRAN_ELEM && c.in_block == 32);
}
// inliers stored as a dense 4-bit operand: no pruning, n:8 / 3:4 sparsification, or element-wise 2:4 with one scale per 32 K
__host__ __device__ inline bool is_dense_layout(const sdq_config_t& c) {
  return c.in_block == 32 && (c.in_gran >= SDQ_GRAN_DENSE || c.in_gran == SDQ_GRAN_ELEM);
}
inline PackedOffsets tiled_offsets(int64_t N, int64_t K, const sdq_config_t& c, bool compact = false) {
  return packed_offsets(N, K, c.out_n, c.in_block == 32, is_dense_layout(c), c.in_gran == SDQ_GRAN_ELEM && c.in_block == 32, compact);
}
// a tiled buffer made by sdq_packed_compact: it has outliers but no container section (its offset, never 0 in a full buffer, is 0)
inline bool is_compact(const sdq_packed_t& p) { return p.cfg.out_n > 0 && p.off[1] == 0; }
inline PackedOffsets tiled_offsets(const sdq_packed_t& p) { return tiled_offsets(p.N, p.K, p.cfg, is_compact(p)); }

struct PlainPackedOffsets {
  size_t in_code, in_meta, in_scale, out_code, out_idx, osexp, total;
};
inline PlainPackedOffsets plain_packed_offsets(int64_t N, int64_t K, const sdq_config_t& c) {
  auto al = [](size_t x) { return (x + 255) & ~(size_t)255; };
  PlainPackedOffsets o;
  const size_t n = (size_t)N, k = (size_t)K;
  o.in_code = 256;
  o.in_meta = al(o.in_code + n * k / 2);
  o.in_scale = al(o.in_meta + n * (c.in_gran == SDQ_GRAN_PAIR ? k / 8 : k / 4));
  o.out_code = al(o.in_scale + n * k / (size_t)c.in_block);
  o.out_idx = al(o.out_code + n * (k / 8) * (size_t)c.out_n);
  o.osexp = al(o.out_idx + n * (k / 8) * (size_t)c.out_n);
  o.total = al(o.osexp + n * 4);
  return o;
}
void launch_pack_plain(const void* W, int64_t N, int64_t K, int64_t ldw, const sdq_config_t& cfg, const float* col_weight, void* buf,
                       uint32_t* flags, cudaStream_t st);
}  // namespace sdq
