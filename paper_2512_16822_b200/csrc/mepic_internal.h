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

// Test hooks for the kernels' give-up paths (see mepic_kernel_test_hooks in mepic.h): the poll limit of every bounded
// wait (the built-in limit when no test changed it) and the index of the one staged copy that is left out (-1: none).
int mepic_test_spin_limit(int built_in);
int mepic_test_skip_tile();
int mepic_test_prefill_two_pass();       // mepic_prefill_test_two_pass: the prefill enqueues its two-pass schedule only

#endif
