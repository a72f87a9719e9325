// Tensor-core (tcgen05) path of the operator.  Placeholder until the kernels land: reports that
// no shape is covered, so every call runs the SIMT kernels.
#pragma once

#include "../../include/rehyat.h"
#include "rehyat_common.cuh"

namespace rehyat {

struct TcWorkspace {};

inline bool tc_shape_supported(bool, int, int, int, int, int, int) { return false; }
inline bool tc_workspace_create(TcWorkspace*, int, int, int, int, size_t* extra) { *extra = 0; return true; }
inline void tc_workspace_destroy(TcWorkspace*) {}
inline int tc_set_attributes() { return REHYAT_OK; }
inline int tc_launch_group(TcWorkspace*, const void*, const void*, const void*, void*, const rehyat_phi_params*,
                           const Geo&, int, int, int, int, int, bool, float*, float*, float*, int, int*,
                           cudaStream_t, int*) {
  return REHYAT_ERR_UNSUPPORTED;
}

}  // namespace rehyat
