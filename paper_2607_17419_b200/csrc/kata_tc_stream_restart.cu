// The streaming chunked kernel over groups of tiles, each restarted from a scanned prefix state (pass 3 of the scan
// forms).  A separate build of the same source.
#define KATA_STREAM_EXPORT 1
#define KATA_STREAM_MODE 2
#include "kata_tc_stream.cu"
