// Host side of the TMA operands: tensor maps for the matrices the tensor-core kernels
// read.  The driver's encoder is looked up through the runtime, so the library does not
// link against the driver library.
#include <cstring>

#include "gsi_umma.cuh"

namespace gsi {

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encoder() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// Row-major bf16 matrix [rows][cols]; boxes of box_rows x 64 elements, 128-byte swizzle.
bool encode(CUtensorMap* m, const void* base, size_t rows, size_t cols, unsigned box_rows) {
  EncodeTiledFn fn = encoder();
  if (!fn || !base) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)umma::kTK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool build_tma_maps(const GroupParams& g, bool front, int max_tokens, TmaMaps* out) {
  std::memset(out, 0, sizeof *out);
  for (int j = 0; j < g.n_maps; ++j)
    if (!encode(&out->w[j], g.W[j], (size_t)g.d_out[j], (size_t)g.d, umma::kTM)) return false;
  const size_t rows = (size_t)front_rows(max_tokens);
  if (!encode(&out->rb, g.rb, 65, (size_t)g.d, umma::kBBox)) return false;
  if (g.flags & GSI_FLAG_DENSE) return true;   // dense baseline: W and bf16(x) in rb only
  if (!front) return true;
  return encode(&out->p, g.P, (size_t)g.d, (size_t)g.k, umma::kTM) &&
         encode(&out->pt, g.PT, (size_t)g.k, (size_t)g.d, umma::kTM) &&
         encode(&out->wp, g.WP, (size_t)g.O, (size_t)g.k, umma::kTM) &&
         encode(&out->xb, g.xb, rows, (size_t)g.d, umma::kBBox) &&
         encode(&out->cb, g.cb, rows, (size_t)g.k, umma::kBBox);
}

}  // namespace gsi
