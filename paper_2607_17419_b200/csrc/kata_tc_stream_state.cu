// The streaming chunked kernel in its state-only form: what a group of tiles adds to the state (pass 1 of the scan
// forms).  A separate build of the same source: no queries, no reads, no intra tile, three key stages.
#define KATA_STREAM_EXPORT 1
#define KATA_STREAM_MODE 3
#include "kata_tc_stream.cu"
