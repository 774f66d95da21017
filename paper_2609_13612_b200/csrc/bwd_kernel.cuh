// Backward kernels (Section 4.4).
#pragma once
#include <cuda.h>
#include "common.cuh"
