// Issue-rate microbenchmark for the roofline of the transforms: eight
// independent chains per thread of one instruction kind each, 2 x 1024
// threads per SM, reported per SM and clock at the nominal maximum clock.
// Integer multiplies, double-precision fused multiply-adds, and both at once
// (odd warps one kind, even warps the other) to see whether the two pipes run
// side by side.
// Standalone program (built by build.py as `int_pipe_bench`); not part of the library.
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#define CHK(x) do{cudaError_t e=(x); if(e){printf("err %s line %d\n", cudaGetErrorString(e), __LINE__); return 1;}}while(0)
template<int MODE> __global__ void k(uint64_t* out, int iters, uint32_t seed) {
  uint32_t a[8]; uint64_t b[8];
  for (int i=0;i<8;i++){ a[i]=threadIdx.x*7+i+seed; b[i]=((uint64_t)a[i]<<32)|(a[i]*2654435761u); }
  double d[8]; for (int i=0;i<8;i++) d[i]=1.0+1e-9*(double)a[i];
  const double dm = 1.0 + 1e-12*(double)seed, dc = 1e-15*(double)seed, dq = 1099510054913.0, dqi = 1.0/dq;
  const bool odd = (threadIdx.x >> 5) & 1;
  uint32_t m = seed|1; uint64_t m64 = ((uint64_t)seed<<33)|0x9E3779B97F4A7C15ull;
  if (MODE==8) {                                          // whole warps of one kind each, no divergence
    if (odd) { for (int it=0; it<iters; it++) {
      #pragma unroll
      for (int i=0;i<8;i++) d[i] = __fma_rn(d[i], dm, dc); } }
    else { for (int it=0; it<iters; it++) {
      #pragma unroll
      for (int i=0;i<8;i++) a[i] = a[i]*m + 12345u; } }
    iters = 0;
  }
  for (int it=0; it<iters; it++) {
    #pragma unroll
    for (int i=0;i<8;i++) {
      if (MODE==0) a[i] = a[i]*m + 12345u;                 // IMAD lo 32
      if (MODE==1) b[i] = (uint64_t)(uint32_t)b[i]*m + b[i];   // IMAD.WIDE
      if (MODE==2) b[i] = __umul64hi(b[i], m64) + 1;       // 64-bit mulhi
      if (MODE==3) b[i] = b[i]*m64 + 1;                    // 64-bit mullo
      if (MODE==4) a[i] = (a[i] + m) ^ (a[i]>>3);          // IADD/LOP/SHF
      if (MODE==9) a[i] = __umulhi(a[i], m) + 12345u;      // IMAD.HI 32
      if (MODE==10) { const uint32_t lo = a[i]*m, hi = __umulhi(a[i], m); a[i] = lo ^ hi; }   // both halves as two narrow multiplies
      if (MODE==11) { const uint64_t p = (uint64_t)a[i]*m; a[i] = (uint32_t)p ^ (uint32_t)(p >> 32); }   // both halves as one wide multiply
      if (MODE==12) { double r; asm("cvt.rni.f64.f64 %0, %1;" : "=d"(r) : "d"(d[i])); d[i] = r + dm; }   // round to integer + DADD
      if (MODE==6) d[i] = __fma_rn(d[i], dm, dc);          // DFMA
      if (MODE==7) {                                        // exact modular product in doubles (6 operations)
        const double y = d[i], w = 123456789012.0;
        const double h = __dmul_rn(y, w), l = __fma_rn(y, w, -h);
        const double kq = __dsub_rn(__fma_rn(h, dqi, 6755399441055744.0), 6755399441055744.0);
        d[i] = __dadd_rn(__fma_rn(-kq, dq, h), l);
      }
      if (MODE==5) { uint64_t hi=__umul64hi(b[i], m64); b[i] = b[i]*0x1234567ull - hi*0xffffffffffc0001ull; } // shoup
    }
  }
  uint64_t s=0; for (int i=0;i<8;i++) s += a[i] + b[i] + (uint64_t)__double_as_longlong(d[i]);
  out[blockIdx.x*blockDim.x+threadIdx.x]=s;
}
template<int MODE> int run(const char* name, double ops_per_iter) {
  int sms; cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0);
  int blocks = sms*2, threads=1024, iters=20000;
  uint64_t* out; CHK(cudaMalloc(&out, (size_t)blocks*threads*8));
  cudaEvent_t e0,e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
  k<MODE><<<blocks,threads>>>(out, 1000, 3); CHK(cudaDeviceSynchronize());
  float best=1e30f;
  for (int r=0;r<3;r++){ cudaEventRecord(e0); k<MODE><<<blocks,threads>>>(out, iters, 3+r); cudaEventRecord(e1); CHK(cudaEventSynchronize(e1)); float ms; cudaEventElapsedTime(&ms,e0,e1); if(ms<best)best=ms; }
  double total = (double)blocks*threads*iters*8*ops_per_iter;
  printf("%-22s %8.3f ms  %10.3f Gop/s  per SM per clk @1.965GHz: %6.1f\n", name, best, total/best/1e6, total/(best*1e-3)/sms/1.965e9);
  cudaFree(out); return 0;
}
int main(){ int sms; cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0); int clk; cudaDeviceGetAttribute(&clk, cudaDevAttrClockRate, 0); printf("SMs %d clock attr %d kHz\n", sms, clk);
  run<0>("imad.lo32",1); run<1>("imad.wide",1); run<2>("umul64hi",1); run<3>("mul.lo.u64",1); run<4>("iadd+lop+shf (3 ops)",3); run<5>("shoup lazy modmul",1);
  run<9>("imad.hi32",1); run<10>("mul.lo + mul.hi pair",1); run<11>("mul.wide, both halves",1); run<12>("cvt.rni.f64 + dadd",1);
  run<6>("dfma",1); run<7>("f64 modmul (6 dp ops)",1); run<8>("imad.lo32 + dfma, alternate warps",1); return 0; }
