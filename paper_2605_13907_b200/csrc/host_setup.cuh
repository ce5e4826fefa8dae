// Host-side set-up shared by the entry points: once-per-device preparation and tensor-map construction.
#pragma once

#include <cuda.h>
#include <stdint.h>

namespace ais {

// Once per device (with that device current): architecture check, kernel attributes, the driver's tensor-map
// encoder.  Returns AIS_OK or AIS_ERR_DEVICE; *num_sms (may be NULL) receives the SM count.
int device_setup(int* num_sms);

// 2-D row-major tensor map (dim0 contiguous).  device_setup() must have succeeded before.
bool make_tmap(CUtensorMap* map, CUtensorMapDataType dtype, const void* base, uint64_t dim0, uint64_t dim1,
               uint64_t stride1_bytes, uint32_t box0, uint32_t box1, CUtensorMapSwizzle swz);

// Bound of the kernels' device-side waits in clock ticks as set by ais_set_wait_cycles (0 = the kernels' default).
int64_t wait_cycles();

}  // namespace ais
