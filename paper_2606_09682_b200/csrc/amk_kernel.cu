// The decode kernel without the trace stamps: the build every step runs unless the handle was created with
// AMK_FLAG_TRACE.
#define AMK_TRACE_BUILD 0
#define AMK_KERNEL amk_decode_kernel
#define AMK_LAUNCH launch_decode
#define AMK_ATTRS decode_kernel_attrs
#include "amk_kernel_impl.cuh"
