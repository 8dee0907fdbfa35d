// Host-callable launchers of the kernels in kernels.cu.
#pragma once
#include <cuda_runtime.h>

#include "device_tables.h"

namespace fmt {

constexpr int SWEEP_WARPS = 24;  // warps of a CTA of the trie sweep: one CTA per SM, so that the grid barrier has few arrivals

cudaError_t configure_kernels();
cudaError_t sweep_blocks_per_sm(int* out, uint32_t smem_bytes);
void sweep_layout(const GrammarDev& G, uint32_t* smem_bytes, uint32_t* tables_in_smem);
int sweep_warps();

void launch_init(const GrammarDev& G, const StateDev& S, int32_t* result_dev, cudaStream_t st);
void launch_intern_init(const StateDev& S, int32_t* init_state_dev, cudaStream_t st);
void launch_reset(const StateDev& S, const uint32_t* rows_dev, uint32_t n, const int32_t* init_state_dev, cudaStream_t st);
void launch_advance(const GrammarDev& G, const StateDev& S, const int32_t* tokens, int32_t* status, cudaStream_t st);
void launch_forced(const GrammarDev& G, const StateDev& S, uint8_t* bytes_out, size_t stride, uint32_t* len_out, uint32_t max_len,
                   cudaStream_t st);
void launch_plan(const GrammarDev& G, const StateDev& S, cudaStream_t st);
void launch_publish(const StateDev& S, cudaStream_t st);
cudaError_t configure_walk_kernels();
void launch_fill(const GrammarDev& G, const StateDev& S, int sweep_grid, cudaStream_t st, cudaEvent_t before_roots = nullptr,
                 cudaEvent_t after_roots = nullptr, cudaEvent_t before_sweep = nullptr, cudaEvent_t after_sweep = nullptr);
void launch_gather(const GrammarDev& G, const StateDev& S, uint32_t* out, size_t stride_words, cudaStream_t st);
void launch_apply(const uint32_t* mask, size_t stride_words, void* logits, int dtype, uint32_t batch, uint32_t V,
                  size_t row_stride, cudaStream_t st);
void launch_gather_apply(const GrammarDev& G, const StateDev& S, void* logits, int dtype, size_t row_stride,
                         uint32_t* mask_out, size_t stride_words, cudaStream_t st);
void launch_evacuate(const StateDev& S, cudaStream_t st);
void launch_survivors(const GrammarDev& G, const StateDev& Old, const StateDev& S, const uint32_t* old_count, cudaStream_t st);
void launch_reintern(const StateDev& S, int32_t* init_state_dev, cudaStream_t st);
void launch_query(const StateDev& S, uint8_t* accepting, uint8_t* finished, uint32_t* n_sets, uint32_t* n_items,
                  int32_t* state_id, cudaStream_t st);

// the trie-walk kernel alone, on an arbitrary grid (used by the allocation-free entry point)
void launch_sweep(const GrammarDev& G, const StateDev& S, int grid, cudaStream_t st);

}  // namespace fmt

struct fmt_grammar;
namespace fmt {
// device tables of a compiled grammar, or nullptr for a host_only grammar; `device` gets its GPU
const GrammarDev* grammar_device_tables(const ::fmt_grammar* g, int* device);
void set_last_error(const char* msg);
}  // namespace fmt
