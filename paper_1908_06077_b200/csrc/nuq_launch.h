// Host-side entry points of the kernel translation units.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "nuq_common.cuh"

namespace nuq {

void build_erc_lut(uint32_t* lut256);                 // ERC(N), N = 1..256: code | len << 16
cudaError_t upload_erc_lut();                         // into the current device's constant memory
cudaError_t launch_bucket_norms(const float* g, uint64_t d, uint32_t bucket, uint32_t norm_kind, float* norms,
                                uint64_t nb, cudaStream_t stream);
size_t encode_smem_bytes(const EncodeParams& P);      // dynamic shared memory of one encoder CTA
int encode_blocks_per_sm(const EncodeParams& P);      // encoder CTAs one SM holds at once (0 on error)
int encode_max_clusters(const EncodeParams& P);       // clusters of P.cluster encoder CTAs the device holds at once (0 on error)
cudaError_t launch_encode(const EncodeParams& P, cudaStream_t stream);
bool fixed4_applies(const Geometry& G);               // the call is served by the 4-bit fixed-width encoder
int fixed4_blocks_per_sm(const EncodeParams& P);
cudaError_t launch_encode_fixed4(const EncodeParams& P, cudaStream_t stream);
cudaError_t launch_level_histogram(const EncodeParams& P, uint64_t* hist, int sms, cudaStream_t stream);   // hist: s + 2 zeroed counters
cudaError_t launch_decode(const DecodeParams& P, int sms, cudaStream_t stream);

}  // namespace nuq
