// Host-side tree / mask descriptor builder and small host utilities.
#include <string.h>

#include "ss_common.cuh"

extern "C" int32_t ss_tree_build(const int32_t* parent, int32_t n_nodes, int32_t gamma, ss_tree_desc* out) {
    if (parent == nullptr || out == nullptr) return SS_ERR_INVALID_ARG;
    if (n_nodes > SS_MAX_NODES || gamma < 0 || gamma > SS_MAX_GAMMA) return SS_ERR_UNSUPPORTED;
    if (n_nodes < 1 || parent[0] != -1) return SS_ERR_BAD_TREE;
    for (int32_t i = 1; i < n_nodes; ++i)
        if (parent[i] < 0 || parent[i] >= i) return SS_ERR_BAD_TREE;
    ss_tree_desc d;
    memset(&d, 0, sizeof d);
    d.n_nodes = n_nodes;
    d.gamma = gamma;
    for (int32_t i = 0; i < SS_MAX_NODES; ++i) d.parent[i] = -1;
    // parent[i] < i, so one ascending sweep extends each parent's finished mask by the node's own bit
    d.anc_mask[0] = 1ull;
    for (int32_t i = 1; i < n_nodes; ++i) {
        const int32_t p = parent[i];
        d.parent[i] = p;
        d.depth[i] = d.depth[p] + 1;
        d.anc_mask[i] = d.anc_mask[p] | (1ull << i);
        if (d.depth[i] > d.max_depth) d.max_depth = d.depth[i];
    }
    *out = d;
    return SS_OK;
}

extern "C" int32_t ss_status(void* workspace, void* stream, int32_t* device_status_out) {
    if (workspace == nullptr || device_status_out == nullptr) return SS_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(s) != cudaSuccess) return SS_ERR_CUDA;
    int32_t v = 0;
    if (cudaMemcpyAsync(&v, workspace, sizeof v, cudaMemcpyDeviceToHost, s) != cudaSuccess) return SS_ERR_CUDA;
    if (cudaMemsetAsync(workspace, 0, sizeof v, s) != cudaSuccess) return SS_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return SS_ERR_CUDA;
    *device_status_out = v;
    return SS_OK;
}

extern "C" int32_t ss_version(void) { return 100; }

extern "C" const char* ss_error_string(int32_t status) {
    switch (status) {
        case SS_OK: return "ok";
        case SS_ERR_INVALID_ARG: return "invalid argument";
        case SS_ERR_BAD_TREE: return "parent array is not a root-first tree";
        case SS_ERR_UNSUPPORTED: return "unsupported shape";
        case SS_ERR_WORKSPACE: return "workspace too small";
        case SS_ERR_CAPACITY: return "sequence exceeds its KV slot capacity";
        case SS_ERR_CUDA: return "CUDA call failed";
        case SS_ERR_DEVICE_TIMEOUT: return "device-side wait ran out";
        default: return "unknown status";
    }
}
