// Programmatic dependent launch: the kernels of one step are launched back to back on one stream, each allowed to
// begin (its CTAs scheduled, its prologue run) while its predecessor is still finishing.
//   pdl_wait():  returns once the preceding kernel of the stream has completed and its writes are visible.  A kernel
//                launched with the programmatic-serialisation attribute must execute it in EVERY CTA before its
//                first access to global memory (reads of the predecessor's results, and writes the predecessor
//                may still be reading), so that "this kernel has completed" keeps implying "everything before it
//                has completed".  Without the attribute it returns at once.
//   pdl_launch_dependents(): this CTA no longer minds the next kernel's CTAs being scheduled beside it; the next
//                kernel starts once every CTA of this one has said so or has exited.
#pragma once

namespace comet {
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
}  // namespace comet
