// Backward kernels of the TSP gated ring MLP.
#pragma once
#include "gemm_core.cuh"
