// Register-resident throughput probes of the inner-product instructions available on sm_100a
// without tensor memory: mma.sync .b1 (and.popc / xor.popc), mma.sync .s8 m16n8k32 and
// CUDA-core xor + popc.  No memory traffic inside the timed loops; prints TMAC/s and TOPS
// (1 MAC = 2 ops).  Build and run:  python -m paper_2010_00704_b200.build --tools
//                                    ./paper_2010_00704_b200/tools/engine_peaks
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#define CK(x) do{cudaError_t e=(x); if(e!=cudaSuccess){printf("ERR %s line %d\n",cudaGetErrorString(e),__LINE__); return 1;}}while(0)

template<int MODE> __global__ void __launch_bounds__(256) k_mma(int iters, int* out, uint32_t seed){
  uint32_t a[4]={seed+threadIdx.x,seed*3+threadIdx.x,seed*5,seed*7}, b0=seed*11+threadIdx.x, b1=seed*13;
  int d[8][4];
  #pragma unroll
  for(int i=0;i<8;i++) for(int j=0;j<4;j++) d[i][j]=0;
  for(int it=0; it<iters; ++it){
    #pragma unroll
    for(int i=0;i<8;i++){
      if(MODE==0) asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[i][0]),"+r"(d[i][1]),"+r"(d[i][2]),"+r"(d[i][3]) : "r"(a[0]),"r"(a[1]),"r"(a[2]),"r"(a[3]),"r"(b0),"r"(b1));
      else if(MODE==1) asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.xor.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[i][0]),"+r"(d[i][1]),"+r"(d[i][2]),"+r"(d[i][3]) : "r"(a[0]),"r"(a[1]),"r"(a[2]),"r"(a[3]),"r"(b0),"r"(b1));
      else asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[i][0]),"+r"(d[i][1]),"+r"(d[i][2]),"+r"(d[i][3]) : "r"(a[0]),"r"(a[1]),"r"(a[2]),"r"(a[3]),"r"(b0),"r"(b1));
    }
  }
  int s=0;
  #pragma unroll
  for(int i=0;i<8;i++) for(int j=0;j<4;j++) s+=d[i][j];
  out[blockIdx.x*blockDim.x+threadIdx.x]=s;
}

__global__ void __launch_bounds__(256) k_popc(int iters, int* out, uint32_t seed){
  uint32_t a[4]={seed+threadIdx.x,seed*3+threadIdx.x,seed*5+blockIdx.x,seed*7};
  uint32_t w[4]={seed*11+threadIdx.x,seed*13,seed*17,seed*19+threadIdx.x};
  int acc[4][4];
  #pragma unroll
  for(int i=0;i<4;i++) for(int j=0;j<4;j++) acc[i][j]=0;
  for(int it=0; it<iters; ++it){
    #pragma unroll
    for(int i=0;i<4;i++)
      #pragma unroll
      for(int j=0;j<4;j++) acc[i][j]+=__popc(a[i]^w[j]);
    #pragma unroll
    for(int i=0;i<4;i++){ a[i]=a[i]*1664525u+1013904223u; }
  }
  int s=0;
  #pragma unroll
  for(int i=0;i<4;i++) for(int j=0;j<4;j++) s+=acc[i][j];
  out[blockIdx.x*blockDim.x+threadIdx.x]=s;
}

int main(){
  int dev=0; cudaDeviceProp pr; CK(cudaGetDeviceProperties(&pr,dev));
  int sms=pr.multiProcessorCount; printf("SMs %d clock %d kHz\n", sms, pr.clockRate);
  int *out; CK(cudaMalloc(&out, sms*8*256*4));
  cudaEvent_t e0,e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
  const char* names[3]={"mma.b1.and k256","mma.b1.xor k256","mma.s8 k32"};
  for(int mode=0; mode<3; ++mode){
    for(int rep=0; rep<3; ++rep){
      int iters=20000; int blocks=sms*4;
      cudaEventRecord(e0);
      if(mode==0) k_mma<0><<<blocks,256>>>(iters,out,12345u);
      else if(mode==1) k_mma<1><<<blocks,256>>>(iters,out,12345u);
      else k_mma<2><<<blocks,256>>>(iters,out,12345u);
      cudaEventRecord(e1); CK(cudaEventSynchronize(e1));
      float ms; cudaEventElapsedTime(&ms,e0,e1);
      double kk = mode<2?256:32;
      double macs=(double)blocks*8*iters*8*16*8*kk;
      printf("%s: %.3f ms  %.1f TMAC/s = %.1f TOPS\n", names[mode], ms, macs/ms/1e9, 2*macs/ms/1e9);
    }
  }
  for(int rep=0; rep<3; ++rep){
    int iters=20000; int blocks=sms*8;
    cudaEventRecord(e0);
    k_popc<<<blocks,256>>>(iters,out,999u);
    cudaEventRecord(e1); CK(cudaEventSynchronize(e1));
    float ms; cudaEventElapsedTime(&ms,e0,e1);
    double macs=(double)blocks*256*iters*16*32;
    printf("popc+xor: %.3f ms  %.1f TMAC/s = %.1f TOPS\n", ms, macs/ms/1e9, 2*macs/ms/1e9);
  }
  CK(cudaDeviceSynchronize());
  return 0;
}
