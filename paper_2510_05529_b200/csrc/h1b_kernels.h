// Launch functions of the H1B-KV kernels (internal to the library).
#pragma once
#include <cuda_runtime.h>

#include "h1b_layout.cuh"

namespace h1b {

// Each launcher enqueues on `st`, adds the number of kernels it launched to
// *launches and returns the launch error, if any.
// Either part may be null: `ap` appends keys/values (and bumps the lengths), `sp` sketches queries.
cudaError_t launch_prepare(const AppendParams *ap, const SketchParams *sp, const NewCounts &nn, cudaStream_t st,
                           int *launches);
// `before` / `after`, when not null, are recorded around the split-K attention kernel alone.
// Long appends: tensor-core projection (Rh holds the two fp16 pieces made by launch_split_projection).
cudaError_t launch_prefill(const PrefillParams &p, const NewCounts &nn, cudaStream_t st, cudaStream_t side,
                           cudaEvent_t fork, cudaEvent_t join, int *launches);
cudaError_t launch_split_projection(const float *Rt, uint16_t *Rh, int n_layers, int m, cudaStream_t st);
cudaError_t launch_decode(const DecodeParams &p, cudaStream_t st, int *launches, cudaEvent_t before = nullptr,
                          cudaEvent_t after = nullptr);
// Sets, on the current device, the launch attributes of every kernel a cache of this shape can reach (thread-safe,
// once per device and kernel): afterwards a launcher only launches.
cudaError_t warm_kernel_attributes(int m_words, int groups, bool paired, bool paged, bool rope);
// Whether the library was compiled with the kernels' index checks (-DH1B_DEBUG_BOUNDS), and a kernel whose one
// check fails on purpose (records its site in *status and skips its store to *target).
bool bounds_checked_build();
cudaError_t launch_debug_bounds_probe(int32_t *status, int32_t *target, cudaStream_t st);
// One warp waits for at most limit_ns on a barrier phase that never completes, then records the time-out in *status.
cudaError_t launch_debug_wait_timeout(int32_t *status, unsigned long long limit_ns, cudaStream_t st);
// Prompt attention on the tensor cores (h1b_prompt.cu): which cache formats it serves, and its launch.
bool prompt_attention_supported(int m_words, int groups, bool paired);
cudaError_t launch_prompt_attention(const PromptParams &p, cudaStream_t st, int *launches, bool attributes_only = false);
cudaError_t launch_set_len(int32_t *len, int n_layers, int max_batch, int seq, int value, cudaStream_t st);
// Scores of key words [w0, w0 + nw) of every cached token of one slab against qwords[0 .. nw).
cudaError_t launch_debug_scores(const CacheAddr &ca, int layer, int b, int kvh, const uint32_t *qwords, int len,
                                int w0, int nw, int32_t *score, cudaStream_t st);

}  // namespace h1b
