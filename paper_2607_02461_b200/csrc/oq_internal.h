// Internal declarations shared by the translation units of liboq (not installed).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <string>
#include <vector>

#include "../../include/oq.h"

struct oq_codebook {
  int dim = 0, bits = 0;
  std::vector<double> centroids;     // 2^bits ascending
  std::vector<double> boundaries;    // 2^bits - 1 midpoints
  std::vector<float> boundaries_f32;
  std::vector<uint16_t> centroids_bf16;
};

struct oq_rpbh {
  int dim = 0, block = 0;
  uint64_t seed = 0;
  std::vector<int32_t> perm;   // (P x)_k = x[perm[k]]
  std::vector<int8_t> signs;   // +1 / -1, indexed by k (after the permutation)
  // device copies, created on first GPU use
  int device = -1;
  uint32_t* d_gather = nullptr;  // [dim] word k: low 16 bits = perm[k], bit 31 = 1 when sign is -1
};

namespace oq {

int fail(int code, const std::string& msg);   // records the message, returns code
int cuda_fail(cudaError_t e, const char* what);
int ensure_device_tables(const oq_rpbh* r);   // uploads d_gather on first use

// Values a kernel needs from a codebook, passed by value as a launch parameter.
struct CodebookParams {
  float pos_bound[8];    // positive boundaries beta_j (j >= 1 of the upper half), unused entries = +inf
  uint16_t level_bf16[16];
  int bits;
};
CodebookParams codebook_params(const oq_codebook* cb);

// Device status word (bounded waits report here).
int* device_status_word();   // device pointer (allocated on first use), or nullptr on failure

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace oq
