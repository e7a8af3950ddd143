// Checked build (-DKVS_DEBUG) of the kernels that apply a sequential rule (dynamic refill, speculative runs):
// every computed index into the caller's profile and per-job outputs and into the warp's working storage is
// tested against its bound before the access.  A violation records (code << 56 | index) in one device word of
// the translation unit - the first one wins - and the access is skipped; nothing traps.  The host reads the
// words through kvs_debug_check_word.  In the normal build KVS_OK_AT is the constant true and costs nothing.
#pragma once

#include "kvs_internal.cuh"

#ifdef KVS_DEBUG
static __device__ unsigned long long g_seq_check_word = 0ull;
__device__ __forceinline__ bool kvs_ok_at(i64 idx, i64 limit, int code) {
  if (idx >= 0 && idx < limit) return true;
  atomicCAS(&g_seq_check_word, 0ull, (static_cast<ull>(code) << 56) | (static_cast<ull>(idx) & 0x00ffffffffffffffull));
  return false;
}
#define KVS_OK_AT(idx, limit, code) kvs_ok_at(static_cast<i64>(idx), static_cast<i64>(limit), (code))
// Host accessor of this translation unit's word.
#define KVS_DEFINE_CHECK_WORD(fn)                                                                       \
  cudaError_t fn(unsigned long long* word, int* compiled, int reset) {                                  \
    if (compiled) *compiled = 1;                                                                        \
    cudaError_t e = cudaMemcpyFromSymbol(word, g_seq_check_word, sizeof(unsigned long long));           \
    if (e == cudaSuccess && reset) {                                                                    \
      const unsigned long long z = 0ull;                                                                \
      e = cudaMemcpyToSymbol(g_seq_check_word, &z, sizeof(z));                                          \
    }                                                                                                   \
    return e;                                                                                           \
  }
#else
#define KVS_OK_AT(idx, limit, code) true
#define KVS_DEFINE_CHECK_WORD(fn)                                                                       \
  cudaError_t fn(unsigned long long* word, int* compiled, int reset) {                                  \
    if (compiled) *compiled = 0;                                                                        \
    *word = 0ull;                                                                                       \
    (void)reset;                                                                                        \
    return cudaSuccess;                                                                                 \
  }
#endif

// codes: refill 32-39, speculative runs 40-49
enum { CHK_RF_JOB = 32, CHK_RF_PROF_OUT = 33, CHK_RF_PROF_WIN = 34, CHK_RF_PROF_IN = 35,
       CHK_SP_LIST = 40, CHK_SP_JOB = 41, CHK_SP_STACK = 42, CHK_SP_PROF = 43, CHK_SP_DROP = 44, CHK_SP_SCRATCH = 45 };
