// Programmatic dependent launch: every kernel of the step is launched with the programmatic stream
// serialization attribute, lets its successor start early (grid_launch_dependents) and itself waits for
// its predecessor to finish and flush (grid_dependency_wait) before it touches global memory.  What
// overlaps is only launch latency and the on-chip prologue (barrier init, tensor-memory allocation,
// descriptor prefetch); all data hazards, read-after-write and write-after-read, are covered because the
// wait is for the full completion of the previous grid.  Without the launch attribute both are no-ops.
#pragma once

namespace jot {
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
}  // namespace jot
