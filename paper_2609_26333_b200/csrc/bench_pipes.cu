// Instruction-throughput micro-benchmarks behind the design of the LUT3 decode kernel (sm_100a).
// Stand-alone program, not part of libdq.so:
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -o bench_pipes bench_pipes.cu && ./bench_pipes
// One CTA per SM, T threads, a loop of independent instructions timed with clock64; prints warp instructions
// per clock per SM for the integer/logic pipe (PRMT, LOP3, SHF), shared-memory lookups (LDS.32 / LDS.64 with
// data-dependent, conflict-free addresses), packed FMAs and mma.sync, and for the inner-loop mixes of the decode
// formulations that were compared (64-bit pair lookup + packed FMA; fp16 pair lookup or register lookup + mma.sync).
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#include <cuda_fp16.h>

#define ITERS 4096
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t c){uint32_t d; asm volatile("prmt.b32 %0,%1,%2,%3;":"=r"(d):"r"(a),"r"(b),"r"(c)); return d;}
__device__ __forceinline__ uint32_t lop3(uint32_t a, uint32_t b, uint32_t c){uint32_t d; asm volatile("lop3.b32 %0,%1,%2,%3,0xCA;":"=r"(d):"r"(a),"r"(b),"r"(c)); return d;}
__device__ __forceinline__ uint32_t shf(uint32_t a, uint32_t n){uint32_t d; asm volatile("shf.r.wrap.b32 %0,%1,%1,%2;":"=r"(d):"r"(a),"r"(n)); return d;}
__device__ __forceinline__ uint32_t lds32(uint32_t a){uint32_t d; asm volatile("ld.shared.u32 %0,[%1];":"=r"(d):"r"(a)); return d;}
__device__ __forceinline__ unsigned long long lds64(uint32_t a){unsigned long long d; asm volatile("ld.shared.u64 %0,[%1];":"=l"(d):"r"(a)); return d;}
__device__ __forceinline__ void ffma2(unsigned long long &acc, unsigned long long a, unsigned long long b){asm volatile("fma.rn.f32x2 %0,%1,%2,%0;":"+l"(acc):"l"(a),"l"(b));}
__device__ __forceinline__ void hfma2(uint32_t &acc, uint32_t a, uint32_t b){asm volatile("fma.rn.f16x2 %0,%1,%2,%0;":"+r"(acc):"r"(a),"r"(b));}
__device__ __forceinline__ void hmul2(uint32_t &d, uint32_t a, uint32_t b){asm volatile("mul.rn.f16x2 %0,%1,%2;":"=r"(d):"r"(a),"r"(b));}
__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0,uint32_t a1,uint32_t a2,uint32_t a3,uint32_t b0,uint32_t b1){
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3},{%4,%5,%6,%7},{%8,%9},{%0,%1,%2,%3};"
   :"+f"(d[0]),"+f"(d[1]),"+f"(d[2]),"+f"(d[3]):"r"(a0),"r"(a1),"r"(a2),"r"(a3),"r"(b0),"r"(b1));}
__device__ __forceinline__ void ffma(float &acc, float a, float b){asm volatile("fma.rn.f32 %0,%1,%2,%0;":"+f"(acc):"f"(a),"f"(b));}

template<int MODE> __global__ void __launch_bounds__(1024,1) k(uint32_t *out, long long *cyc, uint32_t seed)
{
  extern __shared__ uint32_t sm[];
  for (int i=threadIdx.x;i<16384;i+=blockDim.x) sm[i]=i*2654435761u+seed;
  __syncthreads();
  const uint32_t lane=threadIdx.x&31;
  uint32_t r[8]; for(int i=0;i<8;i++) r[i]=seed*(i+3)+threadIdx.x*(2*i+1);
  unsigned long long q[8]; for(int i=0;i<8;i++) q[i]=((unsigned long long)__float_as_uint(1.0f+i)<<32)|__float_as_uint(0.5f*i);
  float d[4][4]={};
  const uint32_t sbase=(uint32_t)__cvta_generic_to_shared(sm);
  long long t0=clock64();
  #pragma unroll 1
  for(int it=0;it<ITERS;++it){
    if (MODE==0){ // PRMT x8 independent chains
      #pragma unroll
      for(int i=0;i<8;i++) r[i]=prmt(r[i],seed,0x3210^i);
    } else if (MODE==1){ // LOP3 x8
      #pragma unroll
      for(int i=0;i<8;i++) r[i]=lop3(r[i],seed,0x0F0F0F0F);
    } else if (MODE==2){ // SHF x8
      #pragma unroll
      for(int i=0;i<8;i++) r[i]=shf(r[i],seed);
    } else if (MODE==3){ // LDS.32 conflict free, address depends on previous result (masked)
      #pragma unroll
      for(int i=0;i<8;i++) r[i]=lds32(sbase + ((r[i]&0xFF)<<7) + lane*4);
    } else if (MODE==4){ // LDS.64 conflict-free
      #pragma unroll
      for(int i=0;i<8;i++){ unsigned long long v=lds64(sbase + ((r[i]&0xFF)<<8) + lane*8); r[i]=(uint32_t)v^(uint32_t)(v>>32);}
    } else if (MODE==5){ // FFMA2 x8
      #pragma unroll
      for(int i=0;i<8;i++) ffma2(q[i],q[(i+1)&7],q[(i+1)&7]);
    } else if (MODE==6){ // HFMA2 x8
      #pragma unroll
      for(int i=0;i<8;i++) hfma2(r[i],r[i],r[i]);
    } else if (MODE==7){ // mma.sync x4 independent accumulators
      #pragma unroll
      for(int i=0;i<4;i++) mma16816(d[i],r[0],r[1],r[2],r[3],r[4],r[5]);
    } else if (MODE==8){ // FFMA x8
      #pragma unroll
      for(int i=0;i<8;i++) ffma(d[i&3][i>>2], d[(i+1)&3][0], 1.0001f);
    } else if (MODE==9){ // per 4 pairs: 8 PRMT + 1 mma (register lookup variant), 4 blocks per iteration
      #pragma unroll
      for(int u=0;u<4;u++){
        uint32_t a[4];
        #pragma unroll
        for(int i=0;i<4;i++){ uint32_t lo=prmt(seed,r[5],r[u]>>(4*i)); uint32_t hi=prmt(r[6],r[7],r[u]>>(4*i)); a[i]=prmt(lo,hi,(i&1)?0x7362:0x5140);} // 12 prmt-ish (shift folded?)
        mma16816(d[u],a[0],a[1],a[2],a[3],r[4],r[5]);
        r[u]=shf(r[u],3);
      }
    } else if (MODE==10){ // per 4 pairs: 4 PRMT + 4 LDS.32 + 1 mma (table lookup variant)
      #pragma unroll
      for(int u=0;u<4;u++){
        uint32_t a[4];
        #pragma unroll
        for(int i=0;i<4;i++){ uint32_t ad=prmt(r[u],sbase+lane*4,0x7604|(i<<4))&0xFFFF; a[i]=lds32(sbase+ad); }
        mma16816(d[u],a[0],a[1],a[2],a[3],r[4],r[5]);
        r[u]=shf(r[u],3);
      }
    } else if (MODE==11){ // current cuda-core: per 4 pairs: 4 PRMT + 4 LDS.64 + 4 FFMA2
      #pragma unroll
      for(int u=0;u<4;u++){
        #pragma unroll
        for(int i=0;i<4;i++){ uint32_t ad=prmt(r[u],sbase+lane*8,0x7604|(i<<4))&0xFFFF; unsigned long long v=lds64(sbase+ad); ffma2(q[i],v,q[4+i]); }
        r[u]=shf(r[u],3);
      }
    } else if (MODE==12){ // per 4 pairs: 2 pairs by registers (4 PRMT) + 2 pairs by table (2 PRMT + 2 LDS.32) + mma
      #pragma unroll
      for(int u=0;u<4;u++){
        uint32_t a[4];
        #pragma unroll
        for(int i=0;i<2;i++){ uint32_t lo=prmt(seed,r[5],r[u]>>(4*i)); uint32_t hi=prmt(r[6],r[7],r[u]>>(4*i)); a[i]=prmt(lo,hi,(i&1)?0x7362:0x5140);}
        #pragma unroll
        for(int i=2;i<4;i++){ uint32_t ad=prmt(r[u],sbase+lane*4,0x7604|(i<<4))&0xFFFF; a[i]=lds32(sbase+ad); }
        mma16816(d[u],a[0],a[1],a[2],a[3],r[4],r[5]);
        r[u]=shf(r[u],3);
      }
    } else if (MODE==14){ // mode 9 without the mma
      #pragma unroll
      for(int u=0;u<4;u++){
        uint32_t a[4];
        #pragma unroll
        for(int i=0;i<4;i++){ uint32_t lo=prmt(seed,r[5],r[u]>>(4*i)); uint32_t hi=prmt(r[6],r[7],r[u]>>(4*i)); a[i]=prmt(lo,hi,(i&1)?0x7362:0x5140);}
        r[4]^=a[0]^a[1]^a[2]^a[3];
        r[u]=shf(r[u],3);
      }
    } else if (MODE==15){ // mode 10 without the mma
      #pragma unroll
      for(int u=0;u<4;u++){
        uint32_t a[4];
        #pragma unroll
        for(int i=0;i<4;i++){ uint32_t ad=prmt(r[u],sbase+lane*4,0x7604|(i<<4))&0xFFFF; a[i]=lds32(sbase+ad); }
        r[4]^=a[0]^a[1]^a[2]^a[3];
        r[u]=shf(r[u],3);
      }
    } else if (MODE==16){ // cvt e2m1x2 -> f16x2, x8
      #pragma unroll
      for(int i=0;i<8;i++){ uint32_t o; asm volatile("{.reg .b8 t; cvt.u8.u32 t, %1; cvt.rn.f16x2.e2m1x2 %0, t;}":"=r"(o):"r"(r[i])); r[i]=o; }
    } else if (MODE==17){ // cvt e4m3x2 -> f16x2, x8
      #pragma unroll
      for(int i=0;i<8;i++){ uint32_t o; asm volatile("cvt.rn.f16x2.e4m3x2 %0, %1;":"=r"(o):"h"((unsigned short)r[i])); r[i]=o; }
    } else if (MODE==18){ // NVFP4 weights to tensor cores: per 4 pairs 4 cvt e2m1x2 + 4 HMUL2 + 1 mma
      #pragma unroll
      for(int u=0;u<4;u++){
        uint32_t a[4];
        #pragma unroll
        for(int i=0;i<4;i++){ uint32_t o; asm volatile("{.reg .b8 t; .reg .b32 w; shr.u32 w, %1, %2; cvt.u8.u32 t, w; cvt.rn.f16x2.e2m1x2 %0, t;}":"=r"(o):"r"(r[u]),"r"(8*i)); hmul2(a[i],o,seed); }
        mma16816(d[u],a[0],a[1],a[2],a[3],r[4],r[5]);
        r[u]=shf(r[u],3);
      }
    } else if (MODE==13){ // HMUL2 x8
      #pragma unroll
      for(int i=0;i<8;i++) hmul2(r[i],r[i],seed);
    }
  }
  long long t1=clock64();
  uint32_t acc=0; for(int i=0;i<8;i++) acc^=r[i]^(uint32_t)q[i]^(uint32_t)(q[i]>>32);
  for(int i=0;i<4;i++) for(int j=0;j<4;j++) acc^=__float_as_uint(d[i][j]);
  out[blockIdx.x*blockDim.x+threadIdx.x]=acc;
  if(threadIdx.x==0) cyc[blockIdx.x]=t1-t0;
}

template<int MODE> void run(const char*name,int ops_per_iter,int threads)
{
  uint32_t*out; long long*cyc; cudaMalloc(&out,148*1024*4); cudaMalloc(&cyc,148*8);
  cudaFuncSetAttribute(k<MODE>,cudaFuncAttributeMaxDynamicSharedMemorySize,65536);
  k<MODE><<<148,threads,65536>>>(out,cyc,12345u); 
  k<MODE><<<148,threads,65536>>>(out,cyc,12345u);
  cudaError_t e=cudaDeviceSynchronize();
  long long h[148]; cudaMemcpy(h,cyc,148*8,cudaMemcpyDeviceToHost);
  double avg=0; for(int i=0;i<148;i++) avg+=h[i]; avg/=148;
  double winst=(double)ITERS*ops_per_iter*(threads/32);
  printf("%-44s thr %4d: %8.0f clk  -> %6.3f warp-instr/clk/SM  (%s)\n",name,threads,avg,winst/avg,cudaGetErrorString(e));
  cudaFree(out); cudaFree(cyc);
}
int main(){
  for(int thr: {512,1024}){
    run<0>("PRMT",8,thr); run<1>("LOP3",8,thr); run<2>("SHF.wrap",8,thr); run<3>("LDS.32 dep",8,thr); run<4>("LDS.64 dep",8,thr);
    run<5>("FFMA2",8,thr); run<6>("HFMA2",8,thr); run<13>("HMUL2",8,thr); run<16>("cvt f16x2.e2m1x2",8,thr); run<17>("cvt f16x2.e4m3x2",8,thr); run<18>("4 cvt.e2m1x2+4 HMUL2+1 mma [4 pairs]",4,thr); run<8>("FFMA",8,thr); run<7>("mma.m16n8k16",4,thr);
    run<9>("reg lookup + mma  [units: 4 pairs]",4,thr); run<14>("reg lookup only [4 pairs]",4,thr); run<10>("4 PRMT+4 LDS32+1 mma [4 pairs]",4,thr); run<15>("4 PRMT+4 LDS32 only [4 pairs]",4,thr);
    run<11>("4 PRMT+4 LDS64+4 FFMA2 [4 pairs]",4,thr); run<12>("half reg / half table + mma [4 pairs]",4,thr);
  }
  return 0;
}
