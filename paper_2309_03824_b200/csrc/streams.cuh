// Streams and events the library owns, for work that runs beside the caller's stream: one set per host thread
// and device, made on that thread's first use (outside any stream capture) and kept until the process exits.  Side work starts after
// the caller's earlier work (fork) and the caller's stream waits for it before the entry point returns (join),
// so to the caller every entry point stays ordered on its own stream, and the pattern can be captured
// into a CUDA graph.  Host threads do not share sets, so calls from different threads do not interfere.
#pragma once
#include "common.cuh"

namespace lrd {

constexpr int kSideStreams = LRD_MAX_GROUP;

struct SideStreams {
    int device = -1;
    cudaStream_t layer[kSideStreams], aux[kSideStreams];       // one per further layer of a group; one per layer for weight gradients
    cudaEvent_t fork, mid, join[kSideStreams], aux_done[kSideStreams];
};

// The calling device's set, or nullptr if it could not be made.
SideStreams* side_streams();

// waiter's next work follows what `done` holds so far
inline bool stream_after(cudaStream_t waiter, cudaStream_t done, cudaEvent_t ev) {
    return cudaEventRecord(ev, done) == cudaSuccess && cudaStreamWaitEvent(waiter, ev, 0) == cudaSuccess;
}

}  // namespace lrd
