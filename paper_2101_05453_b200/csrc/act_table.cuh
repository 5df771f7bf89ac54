// Memoised integer sigmoid / tanh (Section 3.2.1) for the elementwise phase of the persistent recurrent kernel.
//
// The nonlinearities map an int16 to an int16, so a function is fully described by 65 536 values.  Evaluating the
// fixed-point definition (act_q_fast in qmath.cuh: about 45 integer instructions) five times per cell is a third of the
// elementwise phase, which is bound by the integer pipes; a lookup is 7 to 15.  The tables are not a second definition:
// at handle creation a kernel evaluates act_q_fast itself over the whole domain, the host checks the properties the
// compact formats rely on (odd / complementary symmetry, monotone, bounded steps) and packs the values; if any check
// fails the layer simply keeps the arithmetic path.
//
// One blob per layer, three tables, all indexed by a = |x| and holding the quotient q(a) in [0, 32768] of the definition
// before its last step, which is  f(+a) = min(q, 32767)  and  f(-a) = 32768 - q (sigmoid), -q (tanh):
//   sigmoid (gates, Q3.12 in):   plain uint16 [32769]; packed when the plain table would not leave room for the others
//   tanh of the z gate (Q3.12):  packed, see below
//   tanh of the cell (Q_{m.15-m}): the z gate's table when m = 3, else packed when the steps fit, else plain uint16
// Packed format: one 32-bit word per four consecutive inputs 4k .. 4k + 3:
//   bits 0-15 q(4k), bits 16-20 q(4k+1) - q(4k), bits 21-25 q(4k+2) - q(4k), bits 26-30 q(4k+3) - q(4k)
// (offsets from the word's base, not from the previous input, so that decoding is one field extraction).  tanh rises
// by at most 2^m output steps per input step, so the offsets fit 5 bits up to m = 3.
// A table ends at the first input from which on q is constant (tanh reaches 32768 at |x| of about 6); lookups clamp
// |x| to that input.
#pragma once

#include <cstdint>

#include <cuda_runtime.h>

namespace ql {

struct ActTabLayout {
    uint32_t bytes;              // whole blob, a multiple of 16; 0: no tables
    uint32_t tz_off, tc_off;     // byte offsets (multiples of 16) of the two tanh tables; the sigmoid table is at 0
    int32_t tz_amax, tc_amax;    // last |x| with an entry of its own
    int32_t tc_mode;             // cell tanh: 0 the z gate's table, 1 packed, 2 plain uint16
    int32_t sig_packed;          // sigmoid: 0 plain uint16, 1 packed
};

constexpr int ACT_DOMAIN = 32769;                // |x| = 0 .. 32768

// ---- lookups: shared-memory addresses (32 bit) of the tables of one blob ------------------------------------------

struct ActTabs {
    uint32_t sig, tz, tc;        // shared-memory byte addresses
    int32_t tz_amax, tc_amax, tc_mode, sig_packed;
};

__device__ __forceinline__ ActTabs make_act_tabs(uint32_t blob_smem_addr, const ActTabLayout &lay)
{
    ActTabs t;
    t.sig = blob_smem_addr; t.tz = blob_smem_addr + lay.tz_off; t.tc = blob_smem_addr + lay.tc_off;
    t.tz_amax = lay.tz_amax; t.tc_amax = lay.tc_amax; t.tc_mode = lay.tc_mode; t.sig_packed = lay.sig_packed;
    return t;
}

__device__ __forceinline__ uint32_t lds_u16(uint32_t addr)
{
    uint32_t v;
    asm volatile("{ .reg .u16 h; ld.shared.u16 h, [%1]; cvt.u32.u16 %0, h; }" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// q(|x|) of a packed table
__device__ __forceinline__ int32_t packed_q(uint32_t tab, int32_t a)
{
    const uint32_t w = lds_u32(tab + ((uint32_t)a & ~3u));           // word a / 4
    const uint32_t j = (uint32_t)a & 3u;
    const uint32_t off = j ? (w >> (11u + 5u * j)) & 31u : 0u;
    return (int32_t)((w & 0xffffu) + off);
}

__device__ __forceinline__ int32_t tab_packed(uint32_t tab, int32_t amax, int32_t x)
{
    int32_t a = x < 0 ? -x : x;
    a = a < amax ? a : amax;
    const int32_t v = packed_q(tab, a);
    return x < 0 ? -v : (v < 32767 ? v : 32767);
}

__device__ __forceinline__ int32_t tab_sigmoid(const ActTabs &t, int32_t x)
{
    const int32_t a = x < 0 ? -x : x;
    const int32_t v = t.sig_packed ? packed_q(t.sig, a) : (int32_t)lds_u16(t.sig + 2u * (uint32_t)a);
    return x < 0 ? 32768 - v : (v < 32767 ? v : 32767);
}

__device__ __forceinline__ int32_t tab_plain_odd(uint32_t tab, int32_t amax, int32_t x)
{
    int32_t a = x < 0 ? -x : x;
    a = a < amax ? a : amax;
    const int32_t v = (int32_t)lds_u16(tab + 2u * (uint32_t)a);
    return x < 0 ? -v : (v < 32767 ? v : 32767);
}

__device__ __forceinline__ int32_t tab_tanh_gate(const ActTabs &t, int32_t x) { return tab_packed(t.tz, t.tz_amax, x); }

__device__ __forceinline__ int32_t tab_tanh_cell(const ActTabs &t, int32_t x)
{
    return t.tc_mode == 2 ? tab_plain_odd(t.tc, t.tc_amax, x) : tab_packed(t.tc, t.tc_amax, x);
}

// Builds the blob of a layer whose cell state has m_cell integer bits (act_table.cu).  *blob_dev = nullptr and
// lay->bytes = 0 when a check fails or the blob would exceed max_bytes (the caller then keeps the arithmetic path);
// false only on a CUDA error.
bool act_tables_build(int m_cell, size_t max_bytes, uint8_t **blob_dev, ActTabLayout *lay);

}  // namespace ql
