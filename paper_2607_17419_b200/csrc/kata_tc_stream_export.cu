// The streaming chunked kernel with the state hand-off in the public layouts: the state before the first token
// (resume) and after the last token (prefill -> decode).  A separate build of the same source: the plain kernel is
// sensitive to the code the compiler lays around it.
#define KATA_STREAM_EXPORT 1
#define KATA_STREAM_MODE 1
#include "kata_tc_stream.cu"
