// Host utilities: descriptor validation, record size, canonical <-> record repacking, errors.
#include <string.h>

#include "edg_common.cuh"

namespace edg {

static thread_local cudaError_t g_last_error = cudaSuccess;

void set_cuda_error(cudaError_t e) { g_last_error = e; }

static bool pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

int32_t check_desc(const edg_layer_desc* d) {
    if (d == nullptr) return EDG_E_INVAL;
    auto dim_ok = [](int v) { return v >= 128 && v <= 4096 && v % 128 == 0 && pow2(v / 32); };
    if (!dim_ok(d->H) || !dim_ok(d->I)) return EDG_E_SHAPE;
    if (d->group < 32 || d->group % 32 != 0 || d->H % d->group != 0 || d->I % d->group != 0) return EDG_E_SHAPE;
    if ((d->I / kDownSlices) % d->group != 0) return EDG_E_SHAPE;      // a down slice holds whole groups
    if (d->K < 1 || d->K > 32 || d->E < d->K || d->E > 1024) return EDG_E_SHAPE;
    if (d->rank < 0 || d->rank > 64) return EDG_E_SHAPE;
    if (d->n_adapters != 1 && d->n_adapters != d->E) return EDG_E_SHAPE;
    if (d->n_slots < 1) return EDG_E_SHAPE;
    if (d->pre_dtype != EDG_F32 && d->pre_dtype != EDG_F16) return EDG_E_INVAL;
    if (d->out_dtype != EDG_F32 && d->out_dtype != EDG_F16 && d->out_dtype != EDG_BF16) return EDG_E_INVAL;
    return EDG_OK;
}

// interleave (scale, zero) pairs: sz[i] = {scale[i], zero[i]}
static void pack_sz(const uint16_t* s, const uint16_t* z, size_t n, uint8_t* dst) {
    uint16_t* o = reinterpret_cast<uint16_t*>(dst);
    for (size_t i = 0; i < n; ++i) { o[2 * i] = s[i]; o[2 * i + 1] = z[i]; }
}
static void unpack_sz(const uint8_t* src, size_t n, uint16_t* s, uint16_t* z) {
    const uint16_t* o = reinterpret_cast<const uint16_t*>(src);
    for (size_t i = 0; i < n; ++i) { s[i] = o[2 * i]; z[i] = o[2 * i + 1]; }
}

// down: canonical row-major [H][I] <-> kDownSlices column slices
static void pack_down(const edg_layer_desc& d, const RecordLayout& L, const uint8_t* codes, const uint16_t* s,
                      const uint16_t* z, uint8_t* r, bool to_record, uint8_t* codes_out, uint16_t* s_out, uint16_t* z_out) {
    const int H = d.H, I = d.I, g = d.group;
    for (int n = 0; n < H; ++n) {
        for (int c = 0; c < I / 32; ++c) {
            uint8_t* rec = r + L.codes_down + down_code_off(H, I, n, c);
            const size_t can = (size_t)n * (I / 2) + (size_t)c * 16;
            if (to_record) memcpy(rec, codes + can, 16); else memcpy(codes_out + can, rec, 16);
        }
        for (int gi = 0; gi < I / g; ++gi) {
            uint16_t* rec = reinterpret_cast<uint16_t*>(r + L.sz_down + down_sz_off(H, I, g, n, gi));
            const size_t can = (size_t)n * (I / g) + gi;
            if (to_record) { rec[0] = s[can]; rec[1] = z[can]; } else { s_out[can] = rec[0]; z_out[can] = rec[1]; }
        }
    }
}

}  // namespace edg

extern "C" int32_t edg_version(void) { return 1000; }

extern "C" int32_t edg_last_cuda_error(void) { return (int32_t)edg::g_last_error; }

extern "C" const char* edg_last_cuda_error_string(void) { return cudaGetErrorString(edg::g_last_error); }

extern "C" int32_t edg_check_desc(const edg_layer_desc* desc) { return edg::check_desc(desc); }

extern "C" int32_t edg_record_bytes(const edg_layer_desc* desc, size_t* bytes) {
    int32_t rc = edg::check_desc(desc);
    if (rc != EDG_OK) return rc;
    if (!bytes) return EDG_E_INVAL;
    *bytes = edg::record_layout(desc->H, desc->I, desc->group).bytes;
    return EDG_OK;
}

extern "C" int32_t edg_pack_expert(const edg_layer_desc* desc,
                                   const uint8_t* cg, const uint16_t* sg, const uint16_t* zg,
                                   const uint8_t* cu, const uint16_t* su, const uint16_t* zu,
                                   const uint8_t* cd, const uint16_t* sd, const uint16_t* zd, void* record) {
    int32_t rc = edg::check_desc(desc);
    if (rc != EDG_OK) return rc;
    if (!cg || !sg || !zg || !cu || !su || !zu || !cd || !sd || !zd || !record) return EDG_E_INVAL;
    const edg::RecordLayout L = edg::record_layout(desc->H, desc->I, desc->group);
    const size_t cbytes = (size_t)desc->H * desc->I / 2, ngroups = (size_t)desc->H * desc->I / desc->group;
    uint8_t* r = static_cast<uint8_t*>(record);
    // gate / up keep the canonical order (row-major, low nibble first): a 32-bit word then holds
    // code k in bits 4k..4k+3, which is what the in-place nibble masks expect.  down keeps that
    // order inside each of its column slices.
    memcpy(r + L.codes_gate, cg, cbytes);
    memcpy(r + L.codes_up, cu, cbytes);
    edg::pack_sz(sg, zg, ngroups, r + L.sz_gate);
    edg::pack_sz(su, zu, ngroups, r + L.sz_up);
    edg::pack_down(*desc, L, cd, sd, zd, r, true, nullptr, nullptr, nullptr);
    return EDG_OK;
}

extern "C" int32_t edg_unpack_expert(const edg_layer_desc* desc, const void* record,
                                     uint8_t* cg, uint16_t* sg, uint16_t* zg,
                                     uint8_t* cu, uint16_t* su, uint16_t* zu,
                                     uint8_t* cd, uint16_t* sd, uint16_t* zd) {
    int32_t rc = edg::check_desc(desc);
    if (rc != EDG_OK) return rc;
    if (!cg || !sg || !zg || !cu || !su || !zu || !cd || !sd || !zd || !record) return EDG_E_INVAL;
    const edg::RecordLayout L = edg::record_layout(desc->H, desc->I, desc->group);
    const size_t cbytes = (size_t)desc->H * desc->I / 2, ngroups = (size_t)desc->H * desc->I / desc->group;
    const uint8_t* r = static_cast<const uint8_t*>(record);
    memcpy(cg, r + L.codes_gate, cbytes);
    memcpy(cu, r + L.codes_up, cbytes);
    edg::unpack_sz(r + L.sz_gate, ngroups, sg, zg);
    edg::unpack_sz(r + L.sz_up, ngroups, su, zu);
    edg::pack_down(*desc, L, nullptr, nullptr, nullptr, const_cast<uint8_t*>(r), false, cd, sd, zd);
    return EDG_OK;
}
