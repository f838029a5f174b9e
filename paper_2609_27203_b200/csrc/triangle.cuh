// Fused triangle intersect-and-aggregate kernels (filled in below).
#pragma once
#include "engine.cuh"
