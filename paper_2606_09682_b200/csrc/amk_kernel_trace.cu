// The decode kernel with the trace stamps compiled in (AMK_FLAG_TRACE): the same code, a larger instruction
// footprint, a few per cent slower.
#define AMK_TRACE_BUILD 1
#define AMK_KERNEL amk_decode_kernel_traced
#define AMK_LAUNCH launch_decode_traced
#define AMK_ATTRS decode_kernel_attrs_traced
#include "amk_kernel_impl.cuh"
