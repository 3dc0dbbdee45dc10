// Internal declarations shared by the translation units of libmepic (not part of the ABI).
#ifndef MEPIC_INTERNAL_H_
#define MEPIC_INTERNAL_H_

#include "mepic.h"

void mepic_set_error(const char* fmt, ...);
bool mepic_config_ok(const mepic_config_t* cfg);
void mepic_count_launches(int n);
// Fills a 128-byte, 64-byte-aligned CUtensorMap describing a K or V pool (see mepic_tensor_map.cu).
int32_t mepic_make_pool_map(const mepic_config_t* cfg, const void* pool, void* out_map);
int32_t mepic_make_pool_map_u8(const mepic_config_t* cfg, const void* pool, void* out_map);

#endif
