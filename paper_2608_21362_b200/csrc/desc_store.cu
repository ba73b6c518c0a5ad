// Descriptor upload for small and medium calls: the packed tables of one call (chunk, request and
// window descriptors, tensor maps, the attention tile counter) travel as a by-value kernel argument
// and a kernel writes them into the context's device arena.  Compared with a host-to-device copy
// this keeps the call on the compute engine (no copy-engine hand-over in front of the first kernel)
// and, for the stitching calls, the same launch also fills the rotation table (cos / sin of
// delta_pos * theta^(-2j/d), evaluated in double), so the separate table kernel is not needed.
// Two argument sizes: 3840 bytes (inside the classic 4 KB parameter space) and 16384 bytes (the
// parameter space of this architecture holds 32764).  Larger tables go through the pinned staging
// ring and cudaMemcpyAsync.
#include <string.h>

#include "kvb_internal.h"
#include "pdl.cuh"

namespace kvb {
namespace {

template <size_t BYTES>
struct DescBlob {
  uint4 v[BYTES / 16];
};

template <size_t BYTES>
__global__ void __launch_bounds__(128)
    store_blob_kernel(const __grid_constant__ DescBlob<BYTES> blob, int n16, uint4* __restrict__ dst, int n_chunks,
                      const double* __restrict__ inv_freq, int half_d, float2* __restrict__ cs_table) {
  pdl_trigger();  // the call's next kernel may set itself up while this one runs
  pdl_wait();     // the previous call's kernels may still be reading the arena
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n16) dst[i] = blob.v[i];
  if (i < n_chunks * half_d) {  // the chunk descriptors sit at the start of the blob
    const ChunkDesc* cd = reinterpret_cast<const ChunkDesc*>(&blob);
    const int ci = i / half_d, j = i % half_d;
    double sn, cs;
    sincos((double)cd[ci].delta_pos * inv_freq[j], &sn, &cs);
    cs_table[i] = make_float2((float)cs, (float)sn);
  }
}

template <size_t BYTES>
cudaError_t launch_sized(const void* host_bytes, size_t bytes, uint8_t* dst, int n_rope_chunks, const double* inv_freq, int half_d,
                         float2* cs_table, bool pdl, cudaStream_t st) {
  DescBlob<BYTES> blob;
  const size_t padded = (bytes + 15) & ~(size_t)15;
  memcpy(&blob, host_bytes, bytes);
  if (padded > bytes) memset(reinterpret_cast<uint8_t*>(&blob) + bytes, 0, padded - bytes);
  const int n16 = (int)(padded / 16);
  const int work = n16 > n_rope_chunks * half_d ? n16 : n_rope_chunks * half_d;
  return launch_pdl(pdl, store_blob_kernel<BYTES>, dim3((work + 127) / 128), dim3(128), 0, st, blob, n16, reinterpret_cast<uint4*>(dst),
                    n_rope_chunks, inv_freq, half_d, cs_table);
}

}  // namespace

cudaError_t launch_store_blob(const void* host_bytes, size_t bytes, uint8_t* dst, int n_rope_chunks, const double* inv_freq,
                              int half_d, float2* cs_table, bool pdl, cudaStream_t st) {
  if (bytes <= kDescBlobSmall) return launch_sized<kDescBlobSmall>(host_bytes, bytes, dst, n_rope_chunks, inv_freq, half_d, cs_table, pdl, st);
  if (bytes <= kDescBlobBytes) return launch_sized<kDescBlobBytes>(host_bytes, bytes, dst, n_rope_chunks, inv_freq, half_d, cs_table, pdl, st);
  return cudaErrorInvalidValue;
}

}  // namespace kvb
