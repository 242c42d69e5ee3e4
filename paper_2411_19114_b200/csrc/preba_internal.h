// Shared between the host-only and the CUDA translation units of the library.
#ifndef PREBA_INTERNAL_H_
#define PREBA_INTERNAL_H_

#include <stdint.h>

#include "preba.h"

namespace preba {

bool dtype_ok(int out_dtype);
uint32_t dtype_bytes(int out_dtype);  // size of one output element
bool dims_ok(uint32_t h, uint32_t w);
uint64_t align_up(uint64_t v, uint64_t a);

// The cudaError_t behind the calling thread's last PREBA_ERR_CUDA (preba_last_cuda_error).
extern thread_local int g_last_cuda_error;

}  // namespace preba

// The checked build (-DPREBA_CHECKED, a second library built from the same sources): device
// code tests its shared-memory offsets, table indices and global addresses against their
// ranges before it uses them.  A violation stores PREBA_ERR_RANGE in the status word and the
// access is skipped; nothing traps.  In the normal build the test is the constant true and
// costs nothing.  Use: if (PREBA_IN_RANGE(status, index < size)) { ... the access ... }
#if defined(PREBA_CHECKED) && defined(__CUDACC__)
namespace preba {
__device__ __forceinline__ bool range_violation(int32_t* status) {
  if (status) atomicCAS(status, 0, PREBA_ERR_RANGE);
  return false;
}
}  // namespace preba
#define PREBA_IN_RANGE(status, cond) ((cond) ? true : ::preba::range_violation(status))
#else
#define PREBA_IN_RANGE(status, cond) true
#endif

#endif  // PREBA_INTERNAL_H_
