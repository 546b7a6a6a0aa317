// TMA + tcgen05 kernel family (kvc_tc_*.cu): host entry points used by the C ABI.
// Each returns KVC_OK, KVC_E_UNSUPPORTED when the arguments are outside what the
// family serves (the caller then uses the CUDA-core kernels), or another KVC_E_*.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "kvc_dev.cuh"

namespace kvc {

int tc_apply_single(const DevItem& item, int d, int pairing, uint32_t* status, cudaStream_t s, const SegTable* seg = nullptr);
int tc_gate_distance(const DevItem& item, int d, uint32_t* status, double* out, cudaStream_t s);
int tc_row_distance(const DevItem& item, int d, const float* cs2, const float* sn2, uint32_t* status, float* row_out,
                    int64_t t_pad, cudaStream_t s);
int tc_apply_batch(DevItem* tab_host, int64_t* prefix_host, int n_items, int n_table, int d, int pairing, uint32_t* status,
                   void* workspace_dev, void* staging_host, size_t bytes, cudaStream_t s);
size_t tc_batch_extra_bytes(int n_items);
bool tc_batch_item_supported(const DevItem& item, int d);
size_t tc_chain_workspace_bytes(int n_hops, int L, int H);
int tc_chain_fused(const DevItem* items, int n_hops, int d, int pairing, uint32_t* status, void* workspace, size_t ws_bytes,
                   cudaStream_t s);
size_t tc_multi_workspace_bytes(int n_blocks, int L, int H);
int tc_apply_multi(const DevCache& src, const DevCache& dst, int L, int H, int d, const DevState* anchors, int n_anchors,
                   const float* w_k, const float* w_v, int64_t t_pad, int shift, const float* cs, const float* sn, int pairing,
                   uint32_t* status, void* workspace, size_t ws_bytes, cudaStream_t s);
int tc_project(const UpdateLaunch& U, int d, cudaStream_t s);
int tc_gram(const FitLaunch& F, int d, cudaStream_t s, const SegTable* seg = nullptr);
int tc_backproject(const GroupFitLaunch& G, cudaStream_t s, const SegTable* seg = nullptr);

}  // namespace kvc
