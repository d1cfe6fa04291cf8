// Tensor-core (tcgen05 / TMEM) FPROP convolution kernel for sm_100a.
#pragma once
#include "plan.h"
#include "ptx_util.cuh"

namespace maxdnn {
}  // namespace maxdnn
