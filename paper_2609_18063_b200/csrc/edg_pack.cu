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

// canonical row-major [N][Kd] (codes) / [N][Kd/group] (scales, zeros) <-> tile-major sections.
// `down` selects the sliced variant.  to_record: canonical -> record, else record -> canonical.
static void repack(const edg_layer_desc& d, int N, int Kd, bool down, uint8_t* rec_codes, uint8_t* rec_sz,
                   uint8_t* codes, uint16_t* sc, uint16_t* ze, bool to_record) {
    const int g = d.group;
    for (int n = 0; n < N; ++n) {
        for (int c = 0; c < Kd / 32; ++c) {
            uint8_t* r = rec_codes + (down ? down_code_off(d.H, d.I, n, c) : code_off(Kd, n, c));
            uint8_t* k = codes + (size_t)n * (Kd / 2) + (size_t)c * 16;
            if (to_record) memcpy(r, k, 16); else memcpy(k, r, 16);
        }
        for (int gi = 0; gi < Kd / g; ++gi) {
            uint16_t* r = reinterpret_cast<uint16_t*>(rec_sz + (down ? down_sz_off(d.H, d.I, g, n, gi) : sz_off(Kd, g, n, gi)));
            const size_t k = (size_t)n * (Kd / g) + gi;
            if (to_record) { r[0] = sc[k]; r[1] = ze[k]; } else { sc[k] = r[0]; ze[k] = r[1]; }
        }
    }
}

// A zero point the kernels can subtract from a code without rounding: an fp16 value in [0, 16]
// that is a multiple of 1/128 (then q - z, |q - z| <= 16, fits the 11 significant bits of fp16).
static bool zero_point_ok(uint16_t bits) {
    if (bits & 0x8000u) return (bits & 0x7FFFu) == 0;          // -0 only
    const int exp = (bits >> 10) & 0x1F, man = bits & 0x3FF;
    if (exp == 0) return man == 0;                               // subnormals are below 1/128
    if (exp == 0x1F) return false;                               // inf / nan
    const int e = exp - 15;                                      // value = (1024 + man) * 2^(e - 10)
    if (e > 4 || (e == 4 && man != 0)) return false;             // above 16
    const int shift = 3 - e;                                     // low bits that must be clear for a multiple of 2^-7
    if (shift <= 0) return true;
    if (shift > 10) return false;                                // below 1/128 and not zero
    return (man & ((1 << shift) - 1)) == 0;
}

static bool zero_points_ok(const uint16_t* z, size_t n) {
    for (size_t i = 0; i < n; ++i)
        if (!zero_point_ok(z[i])) return false;
    return true;
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
    const size_t n_groups = (size_t)desc->H * desc->I / desc->group;
    if (!edg::zero_points_ok(zg, n_groups) || !edg::zero_points_ok(zu, n_groups) || !edg::zero_points_ok(zd, n_groups))
        return EDG_E_RANGE;
    const edg::RecordLayout L = edg::record_layout(desc->H, desc->I, desc->group);
    uint8_t* r = static_cast<uint8_t*>(record);
    // Inside every 16-byte chunk the canonical nibble order is kept (a 32-bit word holds code k in
    // bits 4k..4k+3); the chunks are re-arranged tile-major.
    edg::repack(*desc, desc->I, desc->H, false, r + L.codes_gate, r + L.sz_gate, const_cast<uint8_t*>(cg),
                const_cast<uint16_t*>(sg), const_cast<uint16_t*>(zg), true);
    edg::repack(*desc, desc->I, desc->H, false, r + L.codes_up, r + L.sz_up, const_cast<uint8_t*>(cu),
                const_cast<uint16_t*>(su), const_cast<uint16_t*>(zu), true);
    edg::repack(*desc, desc->H, desc->I, true, r + L.codes_down, r + L.sz_down, const_cast<uint8_t*>(cd),
                const_cast<uint16_t*>(sd), const_cast<uint16_t*>(zd), true);
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
    const uint8_t* r = static_cast<const uint8_t*>(record);
    uint8_t* rr = const_cast<uint8_t*>(r);
    edg::repack(*desc, desc->I, desc->H, false, rr + L.codes_gate, rr + L.sz_gate, cg, sg, zg, false);
    edg::repack(*desc, desc->I, desc->H, false, rr + L.codes_up, rr + L.sz_up, cu, su, zu, false);
    edg::repack(*desc, desc->H, desc->I, true, rr + L.codes_down, rr + L.sz_down, cd, sd, zd, false);
    return EDG_OK;
}
