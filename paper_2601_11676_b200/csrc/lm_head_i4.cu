// LM-head neuron groups on int4 rows (Sec. II-A, Sec. III-B.3 for the block; Sec. IV-A: the evaluated models are 4-bit).
// Format of halo_quantize_rows_i4: symmetric, one bf16 scale per 128 consecutive elements of a row, nibble = code + 8.
// logits[t][v] = sum over the row's blocks of s_b * sum_e (nibble - 8) * x: a warp takes two vocabulary rows at a time
// against x kept in shared memory in the nibble pairing (nibbles k and k+4 of a word become the bf16 pair
// {128 + n_k, 128 + n_k+4} by mask and OR and feed the mixed-precision FMA; 136 times the plain sum of x over the 32
// elements of a 16-byte chunk is taken off per chunk).  Thread blocks walk (group, 16-row item) pairs in a stride; three
// thread blocks per SM cover each other's loads (holding the next item's rows in registers instead, at two thread blocks
// per SM, was measured slower, and moving a shift to the multiplier and the mask constants into registers, which pays
// in the FFN kernel, changed nothing here: no single pipe is the bound, the issue slots are 55 % busy at 24 warps per SM).
#include <algorithm>

#include "i4_rows.cuh"

namespace halo {

namespace {
constexpr int kLmI4Threads = 256;
constexpr int kLmI4Warps = kLmI4Threads / 32;
constexpr int kLmI4RowsPerItem = 2 * kLmI4Warps;                     // a warp takes two rows of an item
constexpr int kLmI4BlocksPerSm = 3;

__global__ void __launch_bounds__(kLmI4Threads, kLmI4BlocksPerSm)
lm_head_i4_kernel(int d, int vocab, int S, int n_tok, const uint8_t* __restrict__ Q,
                  const __nv_bfloat16* __restrict__ scales, const __nv_bfloat16* __restrict__ x,
                  const int32_t* __restrict__ keep_list, const int32_t* __restrict__ n_keep_ptr,
                  float* __restrict__ logits, uint32_t* dev_status) {
    extern __shared__ __align__(16) unsigned char smem_b[];
    uint4* xp = reinterpret_cast<uint4*>(smem_b);                    // [4][chunks16]: x in nibble pairing
    float* xsum = reinterpret_cast<float*>(smem_b + static_cast<size_t>(d) * 2);   // [chunks16]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_groups = (vocab + S - 1) / S;
    const int items_per_group = (S + kLmI4RowsPerItem - 1) / kLmI4RowsPerItem;
    int nk = n_groups;
    if (keep_list) nk = max(0, min(*n_keep_ptr, n_groups));
    const long long total = static_cast<long long>(nk) * items_per_group;
    // rows of this warp in an item (and whether the item is valid at all)
    auto rows_of = [&](long long item, int& v0, bool& two, bool report) {
        v0 = -1;
        two = false;
        if (item >= total) return;
        const int ki = static_cast<int>(item / items_per_group), rb = static_cast<int>(item - ki * items_per_group);
        const int g = keep_list ? keep_list[ki] : ki;
        if (g < 0 || g >= n_groups) {
            if (report && tid == 0 && rb == 0) flag_status(dev_status, HALO_DEV_BAD_INDEX);
            return;
        }
        const int v_end = min(min(vocab, (g + 1) * S), g * S + (rb + 1) * kLmI4RowsPerItem);
        const int v = g * S + rb * kLmI4RowsPerItem + 2 * warp;
        if (v < v_end) {
            v0 = v;
            two = v + 1 < v_end;
        }
    };
    for (int t = 0; t < n_tok; ++t) {
        if (t > 0) __syncthreads();                                  // everybody is done with the previous x
        stage_x_paired(x + static_cast<size_t>(t) * d, xp, xsum, d);
        __syncthreads();

        for (long long item = blockIdx.x; item < total; item += gridDim.x) {
            int v0;
            bool two;
            rows_of(item, v0, two, t == 0);
            if (v0 >= 0) {                                           // warp-uniform
                float acc_a, acc_b;
                const size_t ra = static_cast<size_t>(v0);           // a lone last row: read twice, used once
                warp_two_rows_dot_i4(Q, scales, ra, two ? ra + 1 : ra, d, xp, xsum, lane, acc_a, acc_b);
                float* out = logits + static_cast<size_t>(t) * vocab + v0;
                if (lane == 0) out[0] = acc_a;
                if (lane == 1 && two) out[1] = acc_b;
            }
        }
    }
}
}  // namespace

}  // namespace halo

using namespace halo;

extern "C" halo_status halo_group_lm_head_i4(const halo_lm_shape* shape, const void* Q, const void* scales, const void* x,
                                             int n_tok, const int32_t* keep_list, const int32_t* n_keep, float* logits,
                                             uint32_t* dev_status, void* stream) {
    if (!shape || !Q || !scales || !x || !logits || !dev_status) return HALO_ERR_ARG;
    if ((keep_list == nullptr) != (n_keep == nullptr)) return HALO_ERR_ARG;
    if (shape->d_model <= 0 || shape->d_model % 128 != 0 || shape->d_model > 8192 || shape->vocab <= 0 ||
        shape->group_size <= 0 || n_tok <= 0)
        return HALO_ERR_SHAPE;
    if (!aligned16(Q) || !aligned16(scales) || !aligned16(x)) return HALO_ERR_ALIGN;
    const int d = shape->d_model, S = shape->group_size;
    const long long n_groups = (static_cast<long long>(shape->vocab) + S - 1) / S;
    const long long items = n_groups * ((S + kLmI4RowsPerItem - 1) / kLmI4RowsPerItem);
    int dev = 0, sms = kSmCount;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const unsigned grid = static_cast<unsigned>(std::min<long long>(items, static_cast<long long>(sms) * kLmI4BlocksPerSm));
    const size_t smem = static_cast<size_t>(d) * 2 + sizeof(float) * (d / 32);
    lm_head_i4_kernel<<<grid, kLmI4Threads, smem, static_cast<cudaStream_t>(stream)>>>(
        d, shape->vocab, S, n_tok, static_cast<const uint8_t*>(Q), static_cast<const __nv_bfloat16*>(scales),
        static_cast<const __nv_bfloat16*>(x), keep_list, n_keep, logits, dev_status);
    return cudaGetLastError() == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}
