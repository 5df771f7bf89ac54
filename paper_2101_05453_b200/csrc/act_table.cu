// Builder of the memoised sigmoid / tanh tables (act_table.cuh): evaluates the fixed-point definitions over the whole
// int16 domain on the device, checks what the compact formats rely on, packs on the host and uploads one blob.
#include <cstring>
#include <vector>

#include <cuda_runtime.h>

#include "act_table.cuh"
#include "qmath.cuh"

namespace ql {

namespace {

// v[f][a] = q(a) for f = sigmoid (m = 3), tanh (m = 3), tanh (m = m_cell), read off the negative side of the definition
// (f(-a) = 32768 - q, -q); *bad != 0 if the positive side is not min(q, 32767)
__global__ void k_act_domain(int m_cell, int32_t *v, int *bad)
{
    const int a = blockIdx.x * blockDim.x + threadIdx.x;
    if (a >= ACT_DOMAIN) return;
    const int32_t sq = 32768 - sigmoid_q_fast(-a, 3), tzq = -tanh_q_fast(-a, 3), tcq = -tanh_q_fast(-a, m_cell);
    v[a] = sq; v[ACT_DOMAIN + a] = tzq; v[2 * ACT_DOMAIN + a] = tcq;
    if (a == 32768) return;                                            // +32768 is not an int16
    const int32_t lim = 32767;
    if (sigmoid_q_fast(a, 3) != (sq < lim ? sq : lim) || tanh_q_fast(a, 3) != (tzq < lim ? tzq : lim) ||
        tanh_q_fast(a, m_cell) != (tcq < lim ? tcq : lim))
        atomicExch(bad, 1);
}

}  // namespace

// ---- host: evaluate on the device, check, pack, upload ------------------------------------------------------------

namespace {

uint32_t pad16(size_t n) { return (uint32_t)((n + 15) & ~(size_t)15); }

// last input with a value of its own: from it on v is constant
int last_own(const int32_t *v)
{
    int a = ACT_DOMAIN - 1;
    while (a > 0 && v[a - 1] == v[a]) --a;
    return a;
}

// packed table of v[0 .. amax]; false if a value or an offset does not fit
bool pack_quads(const int32_t *v, int amax, std::vector<uint32_t> &out)
{
    const int words = amax / 4 + 1;
    out.assign((size_t)words, 0u);
    for (int k = 0; k < words; ++k) {
        const int32_t base = v[4 * k];
        if (base < 0 || base > 0xffff) return false;
        uint32_t w = (uint32_t)base;
        for (int j = 1; j < 4; ++j) {
            const int a = 4 * k + j < ACT_DOMAIN ? 4 * k + j : ACT_DOMAIN - 1;      // past the domain: never looked up
            const int32_t off = v[a] - base;
            if (off < 0 || off > 31) return false;
            w |= (uint32_t)off << (11 + 5 * j);
        }
        out[(size_t)k] = w;
    }
    return true;
}

}  // namespace

bool act_tables_build(int m_cell, size_t max_bytes, uint8_t **blob_dev, ActTabLayout *lay)
{
    *blob_dev = nullptr;
    *lay = ActTabLayout{0, 0, 0, 0, 0, 0, 0};
    int32_t *v_dev = nullptr;
    int *bad_dev = nullptr;
    if (cudaMalloc(&v_dev, 3 * ACT_DOMAIN * sizeof(int32_t)) != cudaSuccess) return false;
    if (cudaMalloc(&bad_dev, sizeof(int)) != cudaSuccess) { cudaFree(v_dev); return false; }
    std::vector<int32_t> v((size_t)3 * ACT_DOMAIN);
    int bad = 0;
    bool ok = cudaMemset(bad_dev, 0, sizeof(int)) == cudaSuccess;
    if (ok) {
        k_act_domain<<<(ACT_DOMAIN + 255) / 256, 256>>>(m_cell, v_dev, bad_dev);
        ok = cudaGetLastError() == cudaSuccess &&
             cudaMemcpy(v.data(), v_dev, v.size() * sizeof(int32_t), cudaMemcpyDeviceToHost) == cudaSuccess &&
             cudaMemcpy(&bad, bad_dev, sizeof(int), cudaMemcpyDeviceToHost) == cudaSuccess;
    }
    cudaFree(v_dev);
    cudaFree(bad_dev);
    if (!ok) return false;
    if (bad) return true;
    const int32_t *sg = v.data(), *tz = sg + ACT_DOMAIN, *tc = tz + ACT_DOMAIN;
    for (int a = 0; a < ACT_DOMAIN; ++a)
        if (sg[a] < 0 || sg[a] > 32768 || tc[a] < 0 || tc[a] > 32768) return true;
    std::vector<uint32_t> tz_words, tc_words;
    const int tz_amax = last_own(tz);
    if (!pack_quads(tz, tz_amax, tz_words)) return true;
    int tc_mode = 0, tc_amax = tz_amax;
    if (m_cell != 3) {
        tc_amax = last_own(tc);
        tc_mode = pack_quads(tc, tc_amax, tc_words) ? 1 : 2;
    }
    // the sigmoid table plain if everything fits then, else packed (its steps are at most 2)
    std::vector<uint32_t> sg_words;
    const size_t tz_bytes = pad16(tz_words.size() * 4);
    const size_t tc_bytes = tc_mode == 0 ? 0 : pad16(tc_mode == 1 ? tc_words.size() * 4 : (size_t)(tc_amax + 1) * 2);
    ActTabLayout L;
    L.sig_packed = 0;
    size_t sg_bytes = pad16((size_t)ACT_DOMAIN * 2);
    if (sg_bytes + tz_bytes + tc_bytes > max_bytes) {
        if (!pack_quads(sg, ACT_DOMAIN - 1, sg_words)) return true;
        L.sig_packed = 1;
        sg_bytes = pad16(sg_words.size() * 4);
    }
    if (sg_bytes + tz_bytes + tc_bytes > max_bytes) return true;
    L.tz_off = (uint32_t)sg_bytes;
    L.tc_off = tc_mode == 0 ? L.tz_off : (uint32_t)(sg_bytes + tz_bytes);
    L.bytes = (uint32_t)(sg_bytes + tz_bytes + tc_bytes);
    L.tz_amax = tz_amax; L.tc_amax = tc_amax; L.tc_mode = tc_mode;
    std::vector<uint8_t> blob((size_t)L.bytes, 0);
    if (L.sig_packed) {
        memcpy(blob.data(), sg_words.data(), sg_words.size() * 4);
    } else {
        uint16_t *s16 = reinterpret_cast<uint16_t *>(blob.data());
        for (int a = 0; a < ACT_DOMAIN; ++a) s16[a] = (uint16_t)sg[a];
    }
    memcpy(blob.data() + L.tz_off, tz_words.data(), tz_words.size() * 4);
    if (tc_mode == 1) memcpy(blob.data() + L.tc_off, tc_words.data(), tc_words.size() * 4);
    if (tc_mode == 2) {
        uint16_t *t16 = reinterpret_cast<uint16_t *>(blob.data() + L.tc_off);
        for (int a = 0; a <= tc_amax; ++a) t16[a] = (uint16_t)tc[a];
    }
    uint8_t *d = nullptr;
    if (cudaMalloc(&d, L.bytes) != cudaSuccess) return false;
    if (cudaMemcpy(d, blob.data(), L.bytes, cudaMemcpyHostToDevice) != cudaSuccess) { cudaFree(d); return false; }
    *blob_dev = d;
    *lay = L;
    return true;
}

}  // namespace ql
