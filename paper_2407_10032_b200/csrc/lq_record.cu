// Storage format of a quantised layer: what the bit columns of the paper's result tables count.
//   non-uniform grid : b-bit codes + one 2^b-entry fp16 table per output row   (b + 16 * 2^b / c bits per weight)
//   affine grid      : b-bit codes + fp16 scale and int16 zero point per group (b + 32 / g bits per weight)
// A record is one device buffer: a 64-byte header, the packed codes (row i is the little-endian bit stream of its
// codes, as lq_pack_codes writes it), then the per-row tables or the per-group parameters.
#include <cuda_fp16.h>

#include "lq_common.cuh"

namespace {

constexpr uint32_t kMagic = 0x3150514cu;      // "LQP1"

struct RecordLayout {
    int64_t row_bytes;       // packed codes per row
    int64_t n_groups;        // affine: groups per row
    size_t codes, table, zero, total;
};

RecordLayout record_layout(const lq_config* cfg, int64_t r, int64_t c) {
    RecordLayout L;
    L.row_bytes = (c * cfg->bits + 7) / 8;
    const int64_t g = cfg->group_size == 0 ? c : cfg->group_size;
    L.n_groups = c / g;
    size_t off = 64;
    L.codes = off; off += lq_align_up(static_cast<size_t>(r) * L.row_bytes, 16);
    if (cfg->grid_type == LQ_GRID_NONUNIFORM) {
        L.table = off; off += lq_align_up(static_cast<size_t>(r) * (size_t(1) << cfg->bits) * 2, 16);
        L.zero = off;
    } else {
        L.table = off; off += lq_align_up(static_cast<size_t>(r) * L.n_groups * 2, 16);
        L.zero = off;  off += lq_align_up(static_cast<size_t>(r) * L.n_groups * 2, 16);
    }
    L.total = off;
    return L;
}

int check_record_cfg(const lq_config* cfg, int64_t r, int64_t c) {
    if (!cfg || r <= 0 || c <= 0) return LQ_ERR_INVALID_ARG;
    if (cfg->bits < 2 || cfg->bits > 4) return LQ_ERR_INVALID_ARG;
    if (cfg->grid_type != LQ_GRID_NONUNIFORM && cfg->grid_type != LQ_GRID_AFFINE) return LQ_ERR_INVALID_ARG;
    if (cfg->grid_type == LQ_GRID_AFFINE) {
        if (cfg->group_size < 0) return LQ_ERR_INVALID_ARG;
        const int64_t g = cfg->group_size == 0 ? c : cfg->group_size;
        if (c % g) return LQ_ERR_INVALID_ARG;
    }
    return LQ_OK;
}

struct Header {
    uint32_t magic;
    int32_t bits, grid_type, group_size;
    long long r, c, codes_offset, table_offset, zero_offset, total_bytes;
};
static_assert(sizeof(Header) == 64, "header is 64 bytes");

__global__ void header_kernel(Header* dst, Header h) { *dst = h; }

// fp16 copies of the per-row tables (non-uniform) or scales (affine); int16 copies of the zero points.
__global__ void to_half_kernel(const float* __restrict__ src, int64_t n, __half* __restrict__ dst) {
    const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i < n) LQ_AT(dst + i) = __float2half_rn(LQ_AT(src + i));
}
__global__ void to_int16_kernel(const int32_t* __restrict__ src, int64_t n, int16_t* __restrict__ dst, lq_dev_status* st) {
    const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i >= n) return;
    int32_t z = LQ_AT(src + i);
    if (z > 32767 || z < -32768) {          // a zero point that 16 bits cannot hold: reported, stored saturated
        lq_report(st, LQ_ERR_UNSUPPORTED, i);
        z = z > 0 ? 32767 : -32768;
    }
    LQ_AT(dst + i) = static_cast<int16_t>(z);
}

// One thread per weight: code from the bit stream, value from the row's table or the group's (S, Z).
template <typename T>
__global__ void unpack_kernel(const uint8_t* __restrict__ rec, int64_t r, int64_t c, int bits, int affine, int64_t group,
                              int64_t n_groups, int64_t row_bytes, size_t off_codes, size_t off_table, size_t off_zero,
                              T* __restrict__ out, int64_t ldo, int check_header, lq_dev_status* st) {
    const int64_t row = blockIdx.y;
    if (check_header && blockIdx.x == 0 && threadIdx.x == 0 && row == 0) {
        const Header* hd = reinterpret_cast<const Header*>(rec);
        if (hd->magic != kMagic || hd->bits != bits || hd->r != r || hd->c != c || hd->grid_type != affine)
            lq_report(st, LQ_ERR_INVALID_ARG, 0);
    }
    const uint8_t* codes = rec + off_codes + row * row_bytes;
    const __half* table = reinterpret_cast<const __half*>(rec + off_table);
    const int16_t* zero = reinterpret_cast<const int16_t*>(rec + off_zero);
    const int K = 1 << bits;
    for (int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; j < c; j += (int64_t)gridDim.x * blockDim.x) {
        const int64_t bit0 = j * bits;
        uint32_t w = LQ_AT(codes + (bit0 >> 3));
        if (((bit0 & 7) + bits > 8) && (bit0 >> 3) + 1 < row_bytes) w |= static_cast<uint32_t>(LQ_AT(codes + (bit0 >> 3) + 1)) << 8;
        const int code = static_cast<int>((w >> (bit0 & 7)) & (K - 1));
        float v;
        if (affine) {
            const int64_t gi = row * n_groups + j / group;
            v = (static_cast<float>(code) - static_cast<float>(LQ_AT(zero + gi))) * __half2float(LQ_AT(table + gi));
        } else {
            v = __half2float(LQ_AT(table + row * K + code));
        }
        LQ_AT(out + row * ldo + j) = T(v);
    }
}

}  // namespace

extern "C" int lq_pack_layer_bytes(const lq_config* cfg, int64_t r, int64_t c, size_t* bytes, double* bits_per_weight) {
    int e = check_record_cfg(cfg, r, c);
    if (e) return e;
    if (!bytes) return LQ_ERR_INVALID_ARG;
    const RecordLayout L = record_layout(cfg, r, c);
    *bytes = L.total;
    if (bits_per_weight) {
        // what the format costs per weight, padding and header left out: the figure the paper's tables print
        const double side = cfg->grid_type == LQ_GRID_NONUNIFORM ? 16.0 * (1 << cfg->bits) / static_cast<double>(c)
                                                                  : 32.0 * L.n_groups / static_cast<double>(c);
        *bits_per_weight = cfg->bits + side;
    }
    return LQ_OK;
}

extern "C" int lq_pack_layer(lq_handle* h, void* stream, const lq_config* cfg, const uint8_t* codes, int64_t r, int64_t c,
                             const float* grid, const float* scale, const int32_t* zero, void* record, size_t record_bytes) {
    int e = check_record_cfg(cfg, r, c);
    if (e) return e;
    if (!h || !codes || !record) return LQ_ERR_INVALID_ARG;
    const bool affine = cfg->grid_type == LQ_GRID_AFFINE;
    if (affine ? (!scale || !zero) : !grid) return LQ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(record) & 15) return LQ_ERR_INVALID_ARG;
    const RecordLayout L = record_layout(cfg, r, c);
    if (record_bytes < L.total) return LQ_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* rec = static_cast<uint8_t*>(record);
    Header hd = {};
    hd.magic = kMagic; hd.bits = cfg->bits; hd.grid_type = cfg->grid_type; hd.group_size = cfg->group_size;
    hd.r = r; hd.c = c;
    hd.codes_offset = static_cast<long long>(L.codes);
    hd.table_offset = static_cast<long long>(L.table);
    hd.zero_offset = static_cast<long long>(L.zero);
    hd.total_bytes = static_cast<long long>(L.total);
    {
        LQ_DBG_SCOPE(h, st);
        LQ_DBG_REG(record, L.total);
        if (grid) LQ_DBG_REG(grid, static_cast<size_t>(r) * (size_t(1) << cfg->bits) * sizeof(float));
        if (affine) LQ_DBG_REG(scale, static_cast<size_t>(r) * L.n_groups * sizeof(float));
        if (affine) LQ_DBG_REG(zero, static_cast<size_t>(r) * L.n_groups * sizeof(int32_t));
        LQ_DBG_COMMIT();
    }
    header_kernel<<<1, 1, 0, st>>>(reinterpret_cast<Header*>(rec), hd);
    LQ_LAUNCH_CHECK();
    e = lq_pack_codes(h, stream, codes, r, c, cfg->bits, rec + L.codes, L.row_bytes);
    if (e) return e;
    if (affine) {
        const int64_t n = r * L.n_groups;
        to_half_kernel<<<static_cast<unsigned>(lq_ceil_div(n, 256)), 256, 0, st>>>(scale, n, reinterpret_cast<__half*>(rec + L.table));
        LQ_LAUNCH_CHECK();
        to_int16_kernel<<<static_cast<unsigned>(lq_ceil_div(n, 256)), 256, 0, st>>>(zero, n, reinterpret_cast<int16_t*>(rec + L.zero),
                                                                                  h->dstatus);
        LQ_LAUNCH_CHECK();
    } else {
        const int64_t n = r * (int64_t(1) << cfg->bits);
        to_half_kernel<<<static_cast<unsigned>(lq_ceil_div(n, 256)), 256, 0, st>>>(grid, n, reinterpret_cast<__half*>(rec + L.table));
        LQ_LAUNCH_CHECK();
    }
    return LQ_OK;
}

extern "C" int lq_unpack_layer(lq_handle* h, void* stream, const lq_config* cfg, const void* record, size_t record_bytes,
                               int64_t r, int64_t c, void* W_hat, int32_t what_dtype, int64_t ldwh) {
    int e = check_record_cfg(cfg, r, c);
    if (e) return e;
    if (!h || !record || !W_hat || ldwh < c || (what_dtype != LQ_F32 && what_dtype != LQ_BF16)) return LQ_ERR_INVALID_ARG;
    const RecordLayout L = record_layout(cfg, r, c);
    if (record_bytes < L.total) return LQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int affine = cfg->grid_type == LQ_GRID_AFFINE ? 1 : 0;
    const int64_t g = cfg->group_size == 0 ? c : cfg->group_size;
    const uint8_t* rec = static_cast<const uint8_t*>(record);
    {
        LQ_DBG_SCOPE(h, st);
        LQ_DBG_REG(record, L.total);
        LQ_DBG_REG(W_hat, (static_cast<size_t>(r - 1) * ldwh + c) * (what_dtype == LQ_F32 ? 4 : 2));
        LQ_DBG_COMMIT();
    }
    for (int64_t r0 = 0; r0 < r; r0 += 65535) {          // rows in slabs: the second grid dimension holds 65535 at most
        const int64_t rr = r - r0 < 65535 ? r - r0 : 65535;
        dim3 grid(static_cast<unsigned>(lq_ceil_div(c, 256) < 64 ? lq_ceil_div(c, 256) : 64), static_cast<unsigned>(rr));
        // the slab's rows start r0 rows into every section; the header check only runs in the first slab
        const size_t oc = L.codes + r0 * L.row_bytes;
        const size_t ot = L.table + r0 * (affine ? L.n_groups : (int64_t(1) << cfg->bits)) * 2;
        const size_t oz = L.zero + r0 * L.n_groups * 2;
        if (what_dtype == LQ_F32)
            unpack_kernel<float><<<grid, 256, 0, st>>>(rec, r, c, cfg->bits, affine, g, L.n_groups, L.row_bytes, oc, ot, oz,
                                                      static_cast<float*>(W_hat) + r0 * ldwh, ldwh, r0 == 0, h->dstatus);
        else
            unpack_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(rec, r, c, cfg->bits, affine, g, L.n_groups, L.row_bytes, oc, ot, oz,
                                                              static_cast<__nv_bfloat16*>(W_hat) + r0 * ldwh, ldwh, r0 == 0, h->dstatus);
        LQ_LAUNCH_CHECK();
    }
    return LQ_OK;
}

// Zeroes the weight columns of input channels that never fired (H_ii = 0), for the layers that share a Hessian with
// the one lq_prepare_hinv was given.  H must still hold the accumulated Hessian (U not aliased onto it).
namespace {
template <typename T>
__global__ void zero_dead_kernel(const float* __restrict__ H, int64_t c, int64_t ldh, T* __restrict__ W, int64_t r, int64_t ldw) {
    const int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (j >= c || LQ_AT(H + j * ldh + j) != 0.0f) return;
    for (int64_t i = blockIdx.y; i < r; i += gridDim.y) LQ_AT(W + i * ldw + j) = T(0.0f);
}
}  // namespace

extern "C" int lq_zero_dead_columns(lq_handle* h, void* stream, const float* H, int64_t c, int64_t ldh, void* W, int32_t w_dtype,
                                    int64_t r, int64_t ldw) {
    if (!h || !H || !W || c <= 0 || r <= 0 || ldh < c || ldw < c || (w_dtype != LQ_F32 && w_dtype != LQ_BF16)) return LQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    {
        LQ_DBG_SCOPE(h, st);
        LQ_DBG_REG(H, (static_cast<size_t>(c - 1) * ldh + c) * sizeof(float));
        LQ_DBG_REG(W, (static_cast<size_t>(r - 1) * ldw + c) * (w_dtype == LQ_F32 ? 4 : 2));
        LQ_DBG_COMMIT();
    }
    dim3 g(static_cast<unsigned>(lq_ceil_div(c, 256)), static_cast<unsigned>(r < 64 ? r : 64));
    if (w_dtype == LQ_F32) zero_dead_kernel<float><<<g, 256, 0, st>>>(H, c, ldh, static_cast<float*>(W), r, ldw);
    else zero_dead_kernel<__nv_bfloat16><<<g, 256, 0, st>>>(H, c, ldh, static_cast<__nv_bfloat16*>(W), r, ldw);
    LQ_LAUNCH_CHECK();
    return LQ_OK;
}
