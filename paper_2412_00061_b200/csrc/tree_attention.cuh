// Parameters shared by the tree-attention kernels.
#pragma once

#include "common.cuh"

namespace ctcsd {

struct AttnParams {
    const void* Q;      // [B,max_nodes,Hq,D]
    const void* K;      // [B,Hkv,Lcap,D]
    const void* V;      // [B,Hkv,Lcap,D]
    void* O;            // [B,max_nodes,Hq,D]
    const int* kv_len;  // [B]
    const int* n_nodes; // [B]
    const unsigned long long* mask;   // [B,max_nodes,ceil(max_nodes/64)]
    int B, Hq, Hkv, D, max_nodes, Lcap;
    float scale;
    int* status;
};

// bf16 on tcgen05 / tensor memory (128-row query tiles; needs Hq/Hkv to divide 128).
bool tree_attention_tc_supported(const AttnParams& p);
int launch_tree_attention_tc(Handle* h, cudaStream_t s, const AttnParams& p);

// bf16 on the warp-level tensor-core instructions (64-row query tiles; any head grouping).
int launch_tree_attention_mma(Handle* h, cudaStream_t s, const AttnParams& p);

// The same kernels with caller-chosen scratch: `part` holds B*Hq*max_nodes*splits*(D+2) floats.
cudaError_t launch_tree_attention_mma_scratch(cudaStream_t s, const AttnParams& p, float* part, int splits);

}  // namespace ctcsd
