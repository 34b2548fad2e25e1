// Varlen scheduler: turns cu_tail_lens into a longest-first request order on the device, so
// that no host synchronisation is needed and long chains start before short ones.
#include "common.cuh"

namespace gdn {

// rank[n] = number of requests that sort before n (longer first, ties by index).  O(N^2 / grid)
// reads of a small array that stays in L1/L2; N is the number of concurrent cache hits.
__global__ void gdn_sched_kernel(const int32_t* __restrict__ cu, int32_t num_seqs,
                                 SchedHeader* header, int32_t* __restrict__ order)
{
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n == 0) header->next_item = 0u;
    if (n >= num_seqs) return;
    const int len_n = cu[n + 1] - cu[n];
    int rank = 0;
    for (int m = 0; m < num_seqs; ++m) {
        const int len_m = cu[m + 1] - cu[m];
        rank += (len_m > len_n) || (len_m == len_n && m < n);
    }
    order[rank] = n;
}

cudaError_t launch_scheduler(const int32_t* cu, int32_t num_seqs, const Sched& s, cudaStream_t stream)
{
    const int threads = 128;
    const int blocks = (num_seqs + threads - 1) / threads;
    gdn_sched_kernel<<<blocks > 0 ? blocks : 1, threads, 0, stream>>>(cu, num_seqs, s.header, s.order);
    return cudaGetLastError();
}

}  // namespace gdn
