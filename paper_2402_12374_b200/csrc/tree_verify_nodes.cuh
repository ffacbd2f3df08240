// What tree_verify.cu and tree_verify_nodes.cu share: the arguments of the verification kernels and the
// node-parallel schedule's host entry points.
#pragma once

#include "common.cuh"

namespace seqtree {

struct VerifyArgs {
  int32_t n, V, slice_cap, flags;
  const int32_t* parent; const int32_t* tokens;
  const float* target; int64_t target_stride;
  const float* draft; int64_t draft_stride;
  float temperature;
  const float* uniforms;
  int32_t* path; int32_t* path_len; int32_t* bonus;
  float* residual_out; int32_t* next_child_out; int32_t* dev_status;
  // batched launch: request r = cluster r; elements between consecutive requests' arrays
  int64_t tree_stride, logits_stride, unif_stride, resid_stride;
};

// Node-parallel schedule (tree_verify_nodes.cu).  Workspace: a few words and two words per node, cleared by the
// launch itself.  `supported` says whether the request fits the schedule at all (vocabulary within what a cluster's
// registers hold, flags it implements).
size_t verify_nodes_workspace_bytes(int n_tree);
bool verify_nodes_supported(int n_tree, int vocab, int flags);
int launch_verify_nodes(const VerifyArgs& a, void* workspace, size_t workspace_bytes, int max_clusters, cudaStream_t stream);

// The walk with rows in registers (tree_verify_walk.cu): one cluster of 16 CTAs, no workspace.
bool verify_walk_supported(int vocab, int flags, float temperature);
// `requests` > 1: a batched launch, one cluster per request (the strides of VerifyArgs lead from one request to the next).
int launch_verify_walk(const VerifyArgs& a, bool check_only, cudaStream_t stream, int requests = 1);

}  // namespace seqtree
