#include "streams.cuh"

namespace lrd {
namespace {
// one table per host thread: calls from different threads never share a stream or an event
thread_local SideStreams g_sides[kMaxDevices];
thread_local int g_n_sides = 0;
}  // namespace

SideStreams* side_streams() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    for (int i = 0; i < g_n_sides; ++i)
        if (g_sides[i].device == dev) return &g_sides[i];
    if (g_n_sides == kMaxDevices) return nullptr;
    SideStreams* ss = &g_sides[g_n_sides];
    bool ok = cudaEventCreateWithFlags(&ss->fork, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&ss->mid, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < kSideStreams && ok; ++i) {
        ok = cudaStreamCreateWithFlags(&ss->layer[i], cudaStreamNonBlocking) == cudaSuccess &&
             cudaStreamCreateWithFlags(&ss->aux[i], cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&ss->join[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&ss->aux_done[i], cudaEventDisableTiming) == cudaSuccess;
    }
    if (!ok) return nullptr;
    ss->device = dev;
    ++g_n_sides;
    return ss;
}

}  // namespace lrd
