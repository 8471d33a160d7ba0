// Pieces shared by the tensor-core attention kernels: PTX wrappers (mbarrier, TMA, tcgen05),
// shared-memory and instruction descriptors, packed fp32 arithmetic, the page resolver of the paged
// key stream, and the host-side tensor-map encoder.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "stages.cuh"

namespace actqkv {
namespace tc {

constexpr uint32_t kSpinLimit = 1u << 24;
// O is rescaled only when a row's maximum grew by more than this (log2 units).  P = 2^(x - m) may
// then reach 2^32: bf16 and fp32 have the range, and the relative precision does not change.
constexpr float kRescaleThreshold = 32.0f;

struct TcParams {
  AttnArgs a;
  int n_q_heads, n_kv_heads, group, block, n_init, n_local_prev, cap_blocks;
  int max_pages, n_phys_pages, n_layers, out_bf16;
  float scale_log2;
  int page_tokens = 16;        // tokens per cache page (the CTA-pair kernel takes 16, 32, 64 or 128)
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the limit expired or another role already gave up.  A phase
// that is already complete (the usual case for operands that arrive tiles ahead) is seen by the
// non-blocking test: try_wait was measured at ~245 cycles per call even then, test_wait at ~30.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          uint32_t limit = kSpinLimit) {
  if (mbar_test_wait(bar, parity)) return true;
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// TMEM loads come with their wait in ONE asm statement, so that no consumer of the registers
// can be scheduled ahead of tcgen05.wait::ld.
#define TMEM_LD64_WAIT(taddr, r) \
  asm volatile( \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%64];\n\t" \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63}, [%65];\n\t" \
      "tcgen05.wait::ld.sync.aligned;" \
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63]) \
      : "r"(taddr), "r"((taddr) + 32) \
      : "memory")
#define TMEM_LD32_WAIT(taddr, r) \
  asm volatile( \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n\t" \
      "tcgen05.wait::ld.sync.aligned;" \
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]) \
      : "r"(taddr) \
      : "memory")
#define TMEM_ST32(taddr, r) \
  asm volatile( \
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" \
      :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]) \
      : "memory")
// 64 columns as 32 register pairs (column 2i in the low half of r[i]), for the packed f32x2 pipe.
#define TMEM_LD64P_WAIT(taddr, r) \
  asm volatile( \
      "{\n\t.reg .b32 t<64>;\n\t" \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {t0,t1,t2,t3,t4,t5,t6,t7,t8,t9,t10,t11,t12,t13,t14,t15,t16,t17,t18,t19,t20,t21,t22,t23,t24,t25,t26,t27,t28,t29,t30,t31}, [%32];\n\t" \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {t32,t33,t34,t35,t36,t37,t38,t39,t40,t41,t42,t43,t44,t45,t46,t47,t48,t49,t50,t51,t52,t53,t54,t55,t56,t57,t58,t59,t60,t61,t62,t63}, [%33];\n\t" \
      "tcgen05.wait::ld.sync.aligned;\n\t" \
      "mov.b64 %0, {t0, t1};\n\t" \
      "mov.b64 %1, {t2, t3};\n\t" \
      "mov.b64 %2, {t4, t5};\n\t" \
      "mov.b64 %3, {t6, t7};\n\t" \
      "mov.b64 %4, {t8, t9};\n\t" \
      "mov.b64 %5, {t10, t11};\n\t" \
      "mov.b64 %6, {t12, t13};\n\t" \
      "mov.b64 %7, {t14, t15};\n\t" \
      "mov.b64 %8, {t16, t17};\n\t" \
      "mov.b64 %9, {t18, t19};\n\t" \
      "mov.b64 %10, {t20, t21};\n\t" \
      "mov.b64 %11, {t22, t23};\n\t" \
      "mov.b64 %12, {t24, t25};\n\t" \
      "mov.b64 %13, {t26, t27};\n\t" \
      "mov.b64 %14, {t28, t29};\n\t" \
      "mov.b64 %15, {t30, t31};\n\t" \
      "mov.b64 %16, {t32, t33};\n\t" \
      "mov.b64 %17, {t34, t35};\n\t" \
      "mov.b64 %18, {t36, t37};\n\t" \
      "mov.b64 %19, {t38, t39};\n\t" \
      "mov.b64 %20, {t40, t41};\n\t" \
      "mov.b64 %21, {t42, t43};\n\t" \
      "mov.b64 %22, {t44, t45};\n\t" \
      "mov.b64 %23, {t46, t47};\n\t" \
      "mov.b64 %24, {t48, t49};\n\t" \
      "mov.b64 %25, {t50, t51};\n\t" \
      "mov.b64 %26, {t52, t53};\n\t" \
      "mov.b64 %27, {t54, t55};\n\t" \
      "mov.b64 %28, {t56, t57};\n\t" \
      "mov.b64 %29, {t58, t59};\n\t" \
      "mov.b64 %30, {t60, t61};\n\t" \
      "mov.b64 %31, {t62, t63};\n\t" \
      "}" \
      : "=l"(r[0]), "=l"(r[1]), "=l"(r[2]), "=l"(r[3]), "=l"(r[4]), "=l"(r[5]), "=l"(r[6]), "=l"(r[7]), "=l"(r[8]), "=l"(r[9]), "=l"(r[10]), "=l"(r[11]), "=l"(r[12]), "=l"(r[13]), "=l"(r[14]), "=l"(r[15]), "=l"(r[16]), "=l"(r[17]), "=l"(r[18]), "=l"(r[19]), "=l"(r[20]), "=l"(r[21]), "=l"(r[22]), "=l"(r[23]), "=l"(r[24]), "=l"(r[25]), "=l"(r[26]), "=l"(r[27]), "=l"(r[28]), "=l"(r[29]), "=l"(r[30]), "=l"(r[31]) \
      : "r"(taddr), "r"((taddr) + 32) \
      : "memory")
// 32 columns as 16 register pairs.
#define TMEM_LD32P_WAIT(taddr, r) \
  asm volatile( \
      "{\n\t.reg .b32 t<32>;\n\t" \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {t0,t1,t2,t3,t4,t5,t6,t7,t8,t9,t10,t11,t12,t13,t14,t15,t16,t17,t18,t19,t20,t21,t22,t23,t24,t25,t26,t27,t28,t29,t30,t31}, [%16];\n\t" \
      "tcgen05.wait::ld.sync.aligned;\n\t" \
      "mov.b64 %0, {t0, t1};\n\t" \
      "mov.b64 %1, {t2, t3};\n\t" \
      "mov.b64 %2, {t4, t5};\n\t" \
      "mov.b64 %3, {t6, t7};\n\t" \
      "mov.b64 %4, {t8, t9};\n\t" \
      "mov.b64 %5, {t10, t11};\n\t" \
      "mov.b64 %6, {t12, t13};\n\t" \
      "mov.b64 %7, {t14, t15};\n\t" \
      "mov.b64 %8, {t16, t17};\n\t" \
      "mov.b64 %9, {t18, t19};\n\t" \
      "mov.b64 %10, {t20, t21};\n\t" \
      "mov.b64 %11, {t22, t23};\n\t" \
      "mov.b64 %12, {t24, t25};\n\t" \
      "mov.b64 %13, {t26, t27};\n\t" \
      "mov.b64 %14, {t28, t29};\n\t" \
      "mov.b64 %15, {t30, t31};\n\t" \
      "}" \
      : "=l"(r[0]), "=l"(r[1]), "=l"(r[2]), "=l"(r[3]), "=l"(r[4]), "=l"(r[5]), "=l"(r[6]), "=l"(r[7]), "=l"(r[8]), "=l"(r[9]), "=l"(r[10]), "=l"(r[11]), "=l"(r[12]), "=l"(r[13]), "=l"(r[14]), "=l"(r[15]) \
      : "r"(taddr) \
      : "memory")
#define TMEM_ST16(taddr, r) \
  asm volatile( \
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" \
      :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) \
      : "memory")
// 16 lanes x 128 columns in the 16x256b shape (verified on the device): thread t, pair 2k + j holds
// lane (t / 4) + 8 j, columns 8 k + 2 (t % 4) and + 1, as one packed register pair.
#define TMEM_LD16X256P_WAIT(taddr, r) \
  asm volatile( \
      "{\n\t.reg .b32 t<64>;\n\t" \
      "tcgen05.ld.sync.aligned.16x256b.x16.b32 {t0,t1,t2,t3,t4,t5,t6,t7,t8,t9,t10,t11,t12,t13,t14,t15,t16,t17,t18,t19,t20,t21,t22,t23,t24,t25,t26,t27,t28,t29,t30,t31,t32,t33,t34,t35,t36,t37,t38,t39,t40,t41,t42,t43,t44,t45,t46,t47,t48,t49,t50,t51,t52,t53,t54,t55,t56,t57,t58,t59,t60,t61,t62,t63}, [%32];\n\t" \
      "tcgen05.wait::ld.sync.aligned;\n\t" \
      "mov.b64 %0, {t0, t1};\n\t" \
      "mov.b64 %1, {t2, t3};\n\t" \
      "mov.b64 %2, {t4, t5};\n\t" \
      "mov.b64 %3, {t6, t7};\n\t" \
      "mov.b64 %4, {t8, t9};\n\t" \
      "mov.b64 %5, {t10, t11};\n\t" \
      "mov.b64 %6, {t12, t13};\n\t" \
      "mov.b64 %7, {t14, t15};\n\t" \
      "mov.b64 %8, {t16, t17};\n\t" \
      "mov.b64 %9, {t18, t19};\n\t" \
      "mov.b64 %10, {t20, t21};\n\t" \
      "mov.b64 %11, {t22, t23};\n\t" \
      "mov.b64 %12, {t24, t25};\n\t" \
      "mov.b64 %13, {t26, t27};\n\t" \
      "mov.b64 %14, {t28, t29};\n\t" \
      "mov.b64 %15, {t30, t31};\n\t" \
      "mov.b64 %16, {t32, t33};\n\t" \
      "mov.b64 %17, {t34, t35};\n\t" \
      "mov.b64 %18, {t36, t37};\n\t" \
      "mov.b64 %19, {t38, t39};\n\t" \
      "mov.b64 %20, {t40, t41};\n\t" \
      "mov.b64 %21, {t42, t43};\n\t" \
      "mov.b64 %22, {t44, t45};\n\t" \
      "mov.b64 %23, {t46, t47};\n\t" \
      "mov.b64 %24, {t48, t49};\n\t" \
      "mov.b64 %25, {t50, t51};\n\t" \
      "mov.b64 %26, {t52, t53};\n\t" \
      "mov.b64 %27, {t54, t55};\n\t" \
      "mov.b64 %28, {t56, t57};\n\t" \
      "mov.b64 %29, {t58, t59};\n\t" \
      "mov.b64 %30, {t60, t61};\n\t" \
      "mov.b64 %31, {t62, t63};\n\t" \
      "}" \
      : "=l"(r[0]), "=l"(r[1]), "=l"(r[2]), "=l"(r[3]), "=l"(r[4]), "=l"(r[5]), "=l"(r[6]), "=l"(r[7]), "=l"(r[8]), "=l"(r[9]), "=l"(r[10]), "=l"(r[11]), "=l"(r[12]), "=l"(r[13]), "=l"(r[14]), "=l"(r[15]), "=l"(r[16]), "=l"(r[17]), "=l"(r[18]), "=l"(r[19]), "=l"(r[20]), "=l"(r[21]), "=l"(r[22]), "=l"(r[23]), "=l"(r[24]), "=l"(r[25]), "=l"(r[26]), "=l"(r[27]), "=l"(r[28]), "=l"(r[29]), "=l"(r[30]), "=l"(r[31]) \
      : "r"(taddr) \
      : "memory")
// 16 lanes x 32 columns in the 16x128b shape: thread t, register 2k + j holds lane (t / 4) + 8 j, column 4 k + (t % 4).
#define TMEM_ST16X128_X8(taddr, r) \
  asm volatile( \
      "tcgen05.st.sync.aligned.16x128b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" \
      :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) \
      : "memory")
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle, version 1 (sm_100).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= uint64_t((saddr & 0x3FFFFu) >> 4);
  d |= uint64_t((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= uint64_t((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= uint64_t(1) << 46;        // descriptor version
  d |= uint64_t(2) << 61;        // SWIZZLE_128B
  return d;
}
// The same descriptor as two 32-bit words, so that the issuing thread advances an operand with one
// 32-bit add on the low word (start address in 16-byte units, no carry into the other fields).
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr, uint32_t lbo_bytes) {
  return ((saddr & 0x3FFFFu) >> 4) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
__host__ __device__ constexpr uint32_t desc_hi(uint32_t sbo_bytes) {
  return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);   // SBO, version 1, SWIZZLE_128B
}
// Instruction descriptor: bf16 x bf16 -> fp32, M x N tile (M = 256 for a CTA pair).
__host__ __device__ constexpr uint32_t make_idesc(bool b_mn_major, int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(b_mn_major) << 16) | (uint32_t(n >> 3) << 17) |
         (uint32_t(m >> 4) << 24);
}
// The same with both operands in fp16 (format code 0 in the A and B fields).
__host__ __device__ constexpr uint32_t make_idesc_f16(bool b_mn_major, int m, int n) {
  return (1u << 4) | (uint32_t(b_mn_major) << 16) | (uint32_t(n >> 3) << 17) | (uint32_t(m >> 4) << 24);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// Saturating form: finite values beyond the fp16 range become +-65504 instead of infinity.
__device__ __forceinline__ uint32_t pack_f16_sat(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// 8 bf16 values (16 bytes) to 8 fp16 values, exact for magnitudes in [2^-14, 65504]; larger finite
// magnitudes saturate at 65504 (an infinity would turn weight-0 products into NaN).
__device__ __forceinline__ uint4 bf16x8_to_f16x8(uint4 v) {
  uint4 r;
  r.x = pack_f16_sat(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u));
  r.y = pack_f16_sat(__uint_as_float(v.y << 16), __uint_as_float(v.y & 0xFFFF0000u));
  r.z = pack_f16_sat(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xFFFF0000u));
  r.w = pack_f16_sat(__uint_as_float(v.w << 16), __uint_as_float(v.w & 0xFFFF0000u));
  return r;
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Packed fp32 pairs (one 64-bit register pair; element 0 in the low half).
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  return (uint64_t(__float_as_uint(hi)) << 32) | __float_as_uint(lo);
}
__device__ __forceinline__ float lo2(uint64_t v) { return __uint_as_float(uint32_t(v)); }
__device__ __forceinline__ float hi2(uint64_t v) { return __uint_as_float(uint32_t(v >> 32)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// (s0, s1) += the two fp16 halves of h2, added in fp32 (mixed-precision add, sm_100).
__device__ __forceinline__ void add_f16x2(float& s0, float& s1, uint32_t h2) {
  asm("{\n\t.reg .f16 a, b;\n\tmov.b32 {a, b}, %2;\n\tadd.rn.f32.f16 %0, a, %0;\n\tadd.rn.f32.f16 %1, b, %1;\n\t}"
      : "+f"(s0), "+f"(s1) : "r"(h2));
}

// Barrier among the kWarps softmax warps that share a TMEM lane quadrant (hardware barrier
// 1 + quadrant; barrier 0 is __syncthreads).  It also ANDs a predicate, so that all of them take
// the same decision to go on or to give up.
template <int kWarps>
__device__ __forceinline__ bool quadrant_sync_and(int quadrant, bool ok) {
  uint32_t res;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %2, 0;\n\t"
      "bar.red.and.pred p, %1, %3, q;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(res) : "r"(quadrant + 1), "r"(uint32_t(ok)), "n"(kWarps * 32) : "memory");
  return res != 0;
}
__device__ __forceinline__ bool pair_sync_and(int quadrant, bool ok) { return quadrant_sync_and<2>(quadrant, ok); }

// Geometry of the key stream of one CTA, shared by the two producer warps.
struct KeyStream {
  const int32_t* sel;
  const int32_t* pt;
  int g_init, g_sel, g_past, gpb, n_cand, n_init, block, max_pages, n_phys_pages, page_base, page_oob;
  int64_t local_start;
};
// Physical page (row of the 4-D tensor map) of 16-token granule gi of the past key stream;
// page_oob (outside the tensor: TMA fills zeros) for padding granules and rejected indices.
__device__ __forceinline__ int granule_page(const KeyStream& ks, int gi, int32_t* status, bool report) {
  if (gi >= ks.g_past) return ks.page_oob;
  int64_t lp;
  if (gi < ks.g_init) {
    lp = gi;
  } else if (gi < ks.g_init + ks.g_sel) {
    const int r = gi - ks.g_init;
    const int blk = ks.sel[r / ks.gpb];
    if (blk < 0 || blk >= ks.n_cand) {
      if (report) set_status(status, ACTQKV_DEV_BAD_SELECTION);
      return ks.page_oob;
    }
    lp = (int64_t(ks.n_init) + int64_t(blk) * ks.block) / 16 + r % ks.gpb;
  } else {
    lp = ks.local_start / 16 + (gi - ks.g_init - ks.g_sel);
  }
  const int phys = lp < ks.max_pages ? ks.pt[lp] : -1;
  if (phys < 0 || phys >= ks.n_phys_pages) {
    if (report) set_status(status, ACTQKV_DEV_BAD_PAGE);
    return ks.page_oob;
  }
  return ks.page_base + phys;
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode() {
  // initialised once, by whichever host thread gets here first (C++11 guarantees the others wait)
  static const EncodeTiledFn fn = [] {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      return reinterpret_cast<EncodeTiledFn>(sym);
    return EncodeTiledFn(nullptr);
  }();
  return fn;
}

// bf16 tensor map with 128-byte swizzle; dims / strides innermost first, strides in bytes (rank - 1 of them).
inline bool encode(CUtensorMap* tm, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides,
            const cuuint32_t* box) {
  EncodeTiledFn fn = get_encode();
  if (!fn) return false;
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


// Tensor map without swizzle for fp32 (fp32 = true) or bf16 data: the box lands in shared memory
// densely, innermost dimension first.
inline bool encode_plain(CUtensorMap* tm, bool fp32, const void* base, int rank, const cuuint64_t* dims,
                         const cuuint64_t* strides, const cuuint32_t* box) {
  EncodeTiledFn fn = get_encode();
  if (!fn) return false;
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(tm, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base),
            dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc
}  // namespace actqkv
