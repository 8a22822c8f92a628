// Many Gossip-PGA iterations of the logistic objective in one launch (narrow states).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "gpga_device.cuh"

namespace gpga {

constexpr uint32_t kLogRunCopyTries = 1u << 18, kLogRunPollTries = 1u << 21;

struct LogRunParams {
    const float* A;       // n x m x d
    const float* y;       // n x m, +-1
    const float* x_in;    // n rows of d floats, row stride ldx: X^(k0)
    float* x_out;         // same layout: receives X^(k0 + steps) (may be x_in)
    long long ldx;
    unsigned long long* ytag;   // logreg_run_ytag_bytes(): published rows and column means, each value paired with its
                                // iteration tag; zero at launch
    int nbuf;             // buffers used in turn (see logreg_run_buffers)
    int* stop;            // one word, zero at launch: set when a bounded wait gave up
    int* error_flag;      // set to 1 if a bounded wait gave up (may be NULL)
    int n, d, m, batch;
    uint32_t k0;          // index of the first iteration
    int steps;            // iterations in this launch
    int topology;         // GPGA_TOPO_RING or GPGA_TOPO_EXP
    int H;                // global average when (k + 1) % H == 0; 0 = never
    int log2n;            // one-peer exponential graph: hops cycle through 2^0 .. 2^(log2n - 1)
    float gamma, l2;
    PhiloxKeys keys;
    // Limits of the kernel's waits: polls of an mbarrier (about 4 us each while incomplete) and reads
    // of a published word (half a microsecond or more each); the defaults make a wait last a second or
    // two before it gives up.  Shorter limits are for the self-test of the give-up path.
    uint32_t copy_tries = kLogRunCopyTries, poll_tries = kLogRunPollTries;
    int launch_nodes = 0;   // > 0: launch only the pairs of nodes 0 .. launch_nodes - 1 (self-test only)
};

// Buffers of half-step rows the kernel cycles through.  A block overwrites the row it published
// nbuf iterations ago, which every reader must have finished with: on the ring and under the global
// average a node cannot publish twice without its readers' rows of the iteration between (two
// buffers); on the one-peer exponential graph the nodes it waits for change with the hop, and a node
// is at most log2 n iterations ahead of any other (log2 n + 2 buffers).
inline int logreg_run_buffers(int topology_is_exp, int log2n) { return topology_is_exp ? log2n + 2 : 2; }
// nbuf row buffers of n x d words, then two buffers of d words for the column means.
inline size_t logreg_run_ytag_bytes(int n, int d, int nbuf)
{
    return ((size_t)nbuf * n * d + 2 * (size_t)d) * sizeof(unsigned long long);
}

// Whether the multi-iteration kernel can take this problem on the current device: ring or one-peer
// exponential topology, d <= 1024, batch <= 128, H < 2^31 and every node's pair of blocks resident
// at the same time.  Returns an error only if a runtime query failed.
cudaError_t logreg_run_supported(int n, int d, int batch, int topology, long long H, bool* ok);

// One launch, `steps` iterations.  p.ytag and p.stop must have been zeroed on the same stream.
cudaError_t launch_logreg_run(const LogRunParams& p, cudaStream_t s);

}  // namespace gpga
