#include "tmap.h"

#include <cudaTypedefs.h>
#include <cuda_runtime.h>

#include <cstring>
#include <list>
#include <vector>

#include "cascade_internal.h"

namespace {

struct Key {
  const void* base;
  uint64_t dims[4];
  uint64_t strides[3];
  uint32_t box[4];
  int rank;
  bool operator==(const Key& o) const { return std::memcmp(this, &o, sizeof(Key)) == 0; }
};

struct Entry {
  Key key;
  alignas(64) CUtensorMap map;
};

// Least recently used first.  A list never moves its elements, so a pointer to a map stays valid until that
// entry is evicted -- and only the entry that has gone unused for longest ever is, thousands of lookups after
// its last use, never one that the call in progress (a dozen maps at most) has fetched.
constexpr size_t kMaxEntries = 4096;
struct Cache {
  std::list<Entry> entries;
};

PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
  }();
  return fn;
}

const CUtensorMap* lookup_or_make(cascade_ctx* ctx, const Key& key) {
  if (ctx->tmap_cache == nullptr) ctx->tmap_cache = new Cache();
  Cache* c = static_cast<Cache*>(ctx->tmap_cache);
  for (auto it = c->entries.begin(); it != c->entries.end(); ++it)
    if (it->key == key) {
      c->entries.splice(c->entries.end(), c->entries, it);  // most recently used last; the element stays where it is in memory
      return &it->map;
    }
  auto fn = encode_fn();
  if (fn == nullptr) return nullptr;
  if (c->entries.size() >= kMaxEntries) c->entries.pop_front();  // callers that churn through buffers
  c->entries.emplace_back();
  Entry& e = c->entries.back();
  std::memset(&e.key, 0, sizeof(Key));
  e.key = key;
  cuuint64_t dims[4], strides[3];
  cuuint32_t box[4], estr[4] = {1, 1, 1, 1};
  for (int i = 0; i < key.rank; ++i) {
    dims[i] = key.dims[i];
    box[i] = key.box[i];
  }
  for (int i = 0; i + 1 < key.rank; ++i) strides[i] = key.strides[i] * 2;  // bytes
  CUresult r = fn(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)key.rank, const_cast<void*>(key.base), dims,
                  strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    c->entries.pop_back();
    return nullptr;
  }
  return &e.map;
}

}  // namespace

const CUtensorMap* get_tmap_2d_bf16(cascade_ctx* ctx, const void* base, uint64_t rows, uint64_t cols,
                                    uint64_t row_stride_elems, uint32_t box_rows, uint32_t box_cols) {
  Key k;
  std::memset(&k, 0, sizeof(k));
  k.base = base;
  k.rank = 2;
  k.dims[0] = cols;
  k.dims[1] = rows;
  k.strides[0] = row_stride_elems;
  k.box[0] = box_cols;
  k.box[1] = box_rows;
  return lookup_or_make(ctx, k);
}

const CUtensorMap* get_tmap_4d_bf16(cascade_ctx* ctx, const void* base, const uint64_t dims[4],
                                    const uint64_t strides_elems[3], const uint32_t box[4]) {
  Key k;
  std::memset(&k, 0, sizeof(k));
  k.base = base;
  k.rank = 4;
  for (int i = 0; i < 4; ++i) {
    k.dims[i] = dims[i];
    k.box[i] = box[i];
  }
  for (int i = 0; i < 3; ++i) k.strides[i] = strides_elems[i];
  return lookup_or_make(ctx, k);
}

const CUtensorMap* get_tmap_bf16(cascade_ctx* ctx, const void* base, int rank, const uint64_t* dims,
                                 const uint64_t* strides_elems, const uint32_t* box) {
  if (rank < 2 || rank > 4) return nullptr;
  Key k;
  std::memset(&k, 0, sizeof(k));
  k.base = base;
  k.rank = rank;
  for (int i = 0; i < rank; ++i) {
    k.dims[i] = dims[i];
    k.box[i] = box[i];
  }
  for (int i = 0; i + 1 < rank; ++i) k.strides[i] = strides_elems[i];
  return lookup_or_make(ctx, k);
}

void free_tmap_cache(cascade_ctx* ctx) {
  delete static_cast<Cache*>(ctx->tmap_cache);
  ctx->tmap_cache = nullptr;
}
