// Device code of the packed aggregation service (umbrella include).
#pragma once

#include "ps_types.cuh"
#include "ps_math.cuh"
#include "ps_kernel_ldg.cuh"
#include "ps_kernel_inline.cuh"
#include "ps_kernel_bulk.cuh"
#include "ps_migrate.cuh"
