// The streaming chunked kernel with the export of the state after the last token (prefill -> decode hand-off).
// A separate build of the same source: the plain kernel is sensitive to the code the compiler lays around it.
#define KATA_STREAM_EXPORT 1
#include "kata_tc_stream.cu"
