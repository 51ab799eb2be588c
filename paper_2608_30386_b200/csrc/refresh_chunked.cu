// Placeholder until the chunked tensor-core kernel lands: reports "no instantiation"
// so that DASC_ALGO_AUTO uses the sequential kernel.
#include "dasc_internal.h"

size_t dasc_refresh_chunked_workspace_bytes(int32_t, int32_t, int32_t) { return 0; }
int dasc_launch_refresh_chunked(const DascRefreshArgs &, void *) { return -1; }
