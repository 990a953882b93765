// Buffer layout of the decompose / quantize-only readings (element-wise 2:4 and / or one scale per 32 K):
// the canonical arrays themselves, one code per byte.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "sdq_internal.h"

namespace sdq {

inline bool is_tensor_core_reading(const sdq_config_t& c) { return c.in_gran == SDQ_GRAN_PAIR && c.in_block == 64; }

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
struct PlainActOffsets {
  size_t xq4_code, xq4_scale, xq8_code, sexp, amax, total;
};
inline PlainActOffsets plain_act_offsets(int64_t M, int64_t K, const sdq_config_t& c) {
  auto al = [](size_t x) { return (x + 255) & ~(size_t)255; };
  PlainActOffsets o;
  const size_t m = (size_t)M, k = (size_t)K;
  o.xq4_code = 0;
  o.xq4_scale = al(o.xq4_code + m * k);
  o.xq8_code = al(o.xq4_scale + m * k / (size_t)c.in_block);
  o.sexp = al(o.xq8_code + m * k);
  o.amax = al(o.sexp + m * 4);
  o.total = al(o.amax + ((m + 7) / 8 * 8) * ((k + 1023) / 1024) * 4);
  return o;
}

void launch_pack_plain(const void* W, int64_t N, int64_t K, int64_t ldw, const sdq_config_t& cfg, const float* col_weight, void* buf,
                       uint32_t* flags, cudaStream_t st);
void launch_quant_plain(const void* X, int64_t M, int64_t K, int64_t ldx, const sdq_config_t& cfg, void* buf, const float* partial,
                        int n_chunks, cudaStream_t st);

}  // namespace sdq
