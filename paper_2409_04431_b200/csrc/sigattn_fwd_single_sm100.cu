// The bf16 forward compiled in its second shape: one 128-row query tile per work item, eight activation
// warps, two thread blocks per SM.  The kernel source is shared with the two-tile shape; see there.
#define SIGATTN_FWD_TILES 1
#include "sigattn_fwd_sm100.cu"
