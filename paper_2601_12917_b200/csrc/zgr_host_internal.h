// Host-side helpers of the context that other translation units of the library may use.
#ifndef ZGR_HOST_INTERNAL_H_
#define ZGR_HOST_INTERNAL_H_

#include <stdint.h>

#include "zgr.h"
#include "zgr_internal.h"

namespace zgr {

PhiloxKeys host_make_keys(uint64_t seed);
NormalScale host_make_scale(double s, int bits);

// Read-only view of a context: descriptor of tensor l (host mirror), mixing scalars, generator mode,
// sticky error code, device ordinal the context is bound to.  Returns false if ctx is null or l is out of range.
bool host_ctx_view(const zgr_ctx* ctx, int32_t l, TensorDesc* desc, double* a, double* b, int* bits, int* sticky, int* device);

}  // namespace zgr
#endif  // ZGR_HOST_INTERNAL_H_
