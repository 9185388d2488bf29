// poss_tree_attention_noalloc: tree-masked attention for callers that cannot allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a region whose memory plan is
// frozen (a serving engine that sized its pools at start-up, a stream-ordered pipeline that must not
// trigger an implicit synchronisation, a plugin that is handed pointers but no allocator).  The regular
// entry point needs a context whose workspace somebody allocated; this one needs nothing but the
// inputs and outputs.  Its split-KV partial results live in a fixed array inside the library image.
#include "poss_internal.cuh"
#include <mutex>

namespace {

// Scratch for the online-softmax partials (m, l, o[d]) of every (row, head, split).  Lives in the
// module's data segment on every GPU that loads the library, until the process exits.
constexpr size_t NOALLOC_SCRATCH_FLOATS = 2u << 20;            // 8 MiB
static __device__ __align__(256) float g_noalloc_scratch[NOALLOC_SCRATCH_FLOATS];

constexpr int MAX_DEVICES = 64;
float* g_scratch_ptr[MAX_DEVICES] = {nullptr};
std::mutex g_setup_mutex;

// The array's name is only a host-side handle; the kernels need its device address, which differs
// per device.  Looked up once per device, with that device current.
int scratch_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return POSS_E_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[dev]) {
    float* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_noalloc_scratch) != cudaSuccess || !p) return POSS_E_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return POSS_OK;
}

}  // namespace

extern "C" POSS_API int poss_tree_attention_noalloc(const void* q, const void* kv, int kv_slots, int prefix_len,
                                                    int rows, int n_q_heads, int n_kv_heads, int head_dim, int dtype,
                                                    const uint64_t* anc_mask, float scale, void* out,
                                                    poss_stream stream) {
  if (!q || !kv || !anc_mask || !out || kv_slots < 1 || prefix_len < 0 || rows < 0) return POSS_E_INVALID;
  if (dtype != POSS_FP32 && dtype != POSS_BF16) return POSS_E_INVALID;
  if (n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads) return POSS_E_SHAPE;
  if (head_dim != 32 && head_dim != 64 && head_dim != 128) return POSS_E_SHAPE;
  int g = n_q_heads / n_kv_heads;
  if (!(g == 1 || g == 2 || g == 3 || g == 4 || g == 8)) return POSS_E_SHAPE;
  // the kernels move keys, values and outputs in 16-byte pieces
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(kv) | reinterpret_cast<uintptr_t>(out)) & 15)
    return POSS_E_INVALID;
  if (((size_t)kv_slots * head_dim * (dtype == POSS_BF16 ? 2 : 4)) & 15) return POSS_E_INVALID;
  if (rows == 0) return POSS_OK;
  if (rows > POSS_MAX_ROWS || prefix_len + rows > kv_slots) return POSS_E_CAPACITY;
  // the fixed scratch bounds the problem: at least one split must fit
  size_t per_split = attn_partial_floats(rows, n_q_heads, head_dim, 1);
  if (per_split > NOALLOC_SCRATCH_FLOATS) return POSS_E_CAPACITY;
  int max_splits = (int)(NOALLOC_SCRATCH_FLOATS / per_split);
  if (max_splits > 32) max_splits = 32;

  float* scratch = nullptr;
  int rc = scratch_for_current_device(&scratch);
  if (rc != POSS_OK) return rc;

  AttnArgs a;
  a.rows = rows; a.Hq = n_q_heads; a.Hkv = n_kv_heads; a.d = head_dim; a.cap = kv_slots;
  a.n_all = prefix_len; a.n_tree = rows; a.mask = anc_mask; a.mask_words = (rows + 63) / 64; a.scale = scale;
  Launcher L;
  L.stream = reinterpret_cast<cudaStream_t>(stream);
  int64_t launches = 0;                     // this call's own count: nothing is shared between callers but the scratch
  L.launches = &launches;
  L.err = POSS_OK;
  size_t half = (size_t)n_kv_heads * kv_slots * head_dim;
  // Nothing in the scratch has to start at zero: every partial that the combine step reads was
  // written by this call's first kernel, so the previous call's leftovers are never seen.
  if (dtype == POSS_BF16) {
    const bf16* kc = reinterpret_cast<const bf16*>(kv);
    run_tree_attention<bf16>(L, a, max_splits, reinterpret_cast<const bf16*>(q), kc, kc + half, scratch,
                             reinterpret_cast<bf16*>(out));
  } else {
    const float* kc = reinterpret_cast<const float*>(kv);
    run_tree_attention<float>(L, a, max_splits, reinterpret_cast<const float*>(q), kc, kc + half, scratch,
                              reinterpret_cast<float*>(out));
  }
  return L.err;
}
