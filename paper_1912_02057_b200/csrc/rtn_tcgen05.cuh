// Thin inline-PTX wrappers for the sm_100a tensor-core path: mbarriers with bounded waits,
// tensor-memory allocation, tcgen05.mma kind::i8 with shared-memory descriptors, tcgen05.ld.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace rtn {
namespace tc {

__device__ __forceinline__ uint32_t smem_addr(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ------------------------------------------------------------------------------------ mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_init_fence()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// One try: the hardware may park the thread for up to `suspend_ns` before answering, so a waiting
// warp does not burn issue slots polling.
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity, uint32_t suspend_ns = 2000)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity), "r"(suspend_ns) : "memory");
    return ok != 0;
}

// Non-blocking test: has the phase of `parity` completed?
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}

// Bounded wait for the phase of `parity` to complete.  After kWaitPolls tries (each parks the thread
// for up to about 2 us: about a second in all) the wait gives up, records it in the status word and
// returns false, so a lost arrival can never hang the GPU.
constexpr uint32_t kWaitPolls = 1u << 19;

__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, unsigned* status,
                                          uint32_t polls = kWaitPolls)
{
    if (mbar_try_wait(bar, parity)) return true;
    for (uint32_t i = 0; i < polls; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
    }
    atomicOr(status, 2u);       // kStatusWaitTimeout
    return false;
}

// ------------------------------------------------------------------------------------ bulk copies
// One contiguous run of global memory -> shared memory, asynchronously; completion is counted in bytes
// on `bar` (no tensor map, no multicast).  Both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst_smem, const void* src, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
// One arrival on `bar` that also announces `bytes` of asynchronous copies to come.
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}

// ------------------------------------------------------------------------------------ launch overlap
// Programmatic dependent launch.  The kernel is launched so that its CTAs may start while the
// previous kernel of the stream is still draining: every access to tensors that kernel may write or read sits behind
// pdl_wait(), which returns once that kernel has completed and its writes are visible; the set-up
// before it reads only the layer's parameters.  pdl_trigger() lets the next kernel of the stream do the same.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ------------------------------------------------------------------------------------ fences
// Shared-memory writes made with ordinary stores become visible to the tensor core (async proxy).
__device__ __forceinline__ void fence_smem_to_async_proxy()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// ------------------------------------------------------------------------------------ tensor memory
// Whole-warp calls.  `cols` is a power of two in [32, 512]; the base address lands in *slot (shared).
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_addr(slot)), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

// ------------------------------------------------------------------------------------ descriptors
// Shared-memory matrix descriptor, K-major operand without swizzle: the operand is a grid of
// "core matrices" of 8 rows x 16 bytes, each stored as 128 contiguous bytes (row r at +16 r).
//   lbo = byte distance between core matrices adjacent along K (next 16 bytes of K)
//   sbo = byte distance between core matrices adjacent along M/N (next 8 rows)
__device__ __forceinline__ uint64_t smem_desc_kmajor(uint32_t saddr, uint32_t lbo, uint32_t sbo)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;                          // descriptor version of sm_100
    return d;                                        // bits 61..63 = 0: no swizzle
}

// Instruction descriptor of tcgen05.mma kind::i8: signed 8-bit A and B, both K-major, int32
// accumulator, dense, D is M x N.
__host__ __device__ constexpr uint32_t idesc_i8(uint32_t M, uint32_t N)
{
    return (2u << 4)            // accumulator format: S32
         | (1u << 7)            // A: signed 8-bit
         | (1u << 10)           // B: signed 8-bit
         | ((N >> 3) << 17)
         | ((M >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem]^T, one K = 32 slice.  Issued by ONE thread.
__device__ __forceinline__ void mma_i8_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                          uint32_t idesc, bool accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate) : "memory");
}

// Same, always accumulating (no predicate set-up in the issue loop).
__device__ __forceinline__ void mma_i8_ss_acc(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.eq.b32 p, 0, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc) : "memory");
}

// Makes `bar` receive one arrival once every tcgen05.mma this thread issued so far has finished.
__device__ __forceinline__ void mma_commit(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(smem_addr(bar)) : "memory");
}

// Each lane of the warp reads 16 consecutive 32-bit columns of its own TMEM lane
// (warp w may touch lanes 32 (w mod 4) .. +31 only).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
          "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
// Eight columns per lane.
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&v)[8])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
        : "r"(taddr) : "memory");
}

// Each lane writes 16 consecutive 32-bit columns of its own TMEM lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ------------------------------------------------------------------------------------ unpack
// 32 ternary codes given as one word of plane 1 (non-zero) and one of plane 2 (sign) -> 32 int8
// values {0, +1, -1} in eight 32-bit words.  Two-bit codes (plane-2 bit, plane-1 bit) index a
// four-entry byte table through PRMT: 00 -> 0, 01 -> -1, 10 -> 0 (the second zero of Table 1),
// 11 -> +1.  Output byte order (k = code index 0..31): word 0 holds k = 0,4,8,12; word 1 k =
// 2,6,10,14; word 2 k = 1,5,9,13; word 3 k = 3,7,11,15; words 4..7 the same plus 16.  Both GEMM
// operands go through this function, so the order cancels in the dot product.
__device__ __forceinline__ void unpack32(uint32_t nz, uint32_t sg, uint32_t (&o)[8])
{
    constexpr uint32_t kTable = 0x0100FF00u;       // byte[index]: 0, -1, 0, +1
    const uint32_t q = (nz & 0x55555555u) | ((sg << 1) & 0xAAAAAAAAu);       // codes of even k
    const uint32_t r = ((nz >> 1) & 0x55555555u) | (sg & 0xAAAAAAAAu);       // codes of odd k
    const uint32_t q0 = q & 0x33333333u, q1 = (q >> 2) & 0x33333333u;
    const uint32_t r0 = r & 0x33333333u, r1 = (r >> 2) & 0x33333333u;
    o[0] = __byte_perm(kTable, kTable, q0);
    o[1] = __byte_perm(kTable, kTable, q1);
    o[2] = __byte_perm(kTable, kTable, r0);
    o[3] = __byte_perm(kTable, kTable, r1);
    o[4] = __byte_perm(kTable, kTable, q0 >> 16);
    o[5] = __byte_perm(kTable, kTable, q1 >> 16);
    o[6] = __byte_perm(kTable, kTable, r0 >> 16);
    o[7] = __byte_perm(kTable, kTable, r1 >> 16);
}

// Half of unpack32: codes 16*half .. 16*half+15 of the word pair -> four words (one 16-byte chunk),
// same byte order as words 4*half .. 4*half+3 of unpack32.
__device__ __forceinline__ void unpack16(uint32_t nz, uint32_t sg, int half, uint32_t (&o)[4])
{
    constexpr uint32_t kTable = 0x0100FF00u;
    const uint32_t q = (nz & 0x55555555u) | ((sg << 1) & 0xAAAAAAAAu);
    const uint32_t r = ((nz >> 1) & 0x55555555u) | (sg & 0xAAAAAAAAu);
    const int sh = 16 * half;
    o[0] = __byte_perm(kTable, kTable, (q & 0x33333333u) >> sh);
    o[1] = __byte_perm(kTable, kTable, ((q >> 2) & 0x33333333u) >> sh);
    o[2] = __byte_perm(kTable, kTable, (r & 0x33333333u) >> sh);
    o[3] = __byte_perm(kTable, kTable, ((r >> 2) & 0x33333333u) >> sh);
}

}  // namespace tc
}  // namespace rtn
