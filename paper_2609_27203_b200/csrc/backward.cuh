// Gradient kernels of logsumexp / sum rules (filled in below).
#pragma once
#include "engine.cuh"
