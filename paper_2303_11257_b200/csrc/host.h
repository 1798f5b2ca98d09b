// Host-side helpers shared by the translation units of libunitscale.
#pragma once
#include <cuda_runtime.h>

#include "../../include/unitscale.h"

namespace us {
namespace host {
// Number of SMs of the current device (cached per device), or -1 on error.
int sm_count();
}  // namespace host
}  // namespace us
