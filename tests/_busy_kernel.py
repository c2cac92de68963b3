"""A kernel for a second stream that keeps the load/store units of the SMs busy: every thread sums rows of 16-byte loads
that lie 512 bytes apart, the access pattern of a per-row reduction over a [rows, 256] bf16 array.  Compiled at run time with
NVRTC (cuda-python) to PTX and launched through the driver API on a torch stream, so that tests can run the library's
kernels with other work resident on the same SMs.  Test infrastructure only."""
import ctypes

import torch

_SRC = r"""
extern "C" __global__ void __launch_bounds__(128)
busy_rows(const uint4 *__restrict__ src, int rows, int row_u4, int reps, float *sink) {
    const int r0 = blockIdx.x * 128 + threadIdx.x;
    float s = 0.f;
    for (int k = 0; k < reps; ++k) {
        const int r = (int)(((long long)r0 + (long long)k * 9973) % rows);
        const uint4 *p = src + (size_t)r * row_u4;
        for (int i = 0; i < row_u4; ++i) {
            const uint4 v = __ldg(p + i);
            s += __uint_as_float(v.x) + __uint_as_float(v.y) + __uint_as_float(v.z) + __uint_as_float(v.w);
        }
    }
    if (s == 1.2345e-30f) *sink = s;          // never true for the data used: keeps the loads alive, writes nothing
}
"""


class BusyKernel:
    def __init__(self, device="cuda:0", rows=1 << 16, row_bytes=512):
        from cuda.bindings import driver, nvrtc
        self.driver = driver
        torch.cuda.init()
        torch.zeros(1, device=device)                         # makes the primary context current
        err, prog = nvrtc.nvrtcCreateProgram(_SRC.encode(), b"busy_rows.cu", 0, [], [])
        assert err == nvrtc.nvrtcResult.NVRTC_SUCCESS, err
        opts = [b"--gpu-architecture=compute_100", b"-default-device"]
        err, = nvrtc.nvrtcCompileProgram(prog, len(opts), opts)
        if err != nvrtc.nvrtcResult.NVRTC_SUCCESS:
            _, n = nvrtc.nvrtcGetProgramLogSize(prog)
            log = b" " * n
            nvrtc.nvrtcGetProgramLog(prog, log)
            raise RuntimeError(log.decode(errors="replace"))
        _, n = nvrtc.nvrtcGetPTXSize(prog)
        ptx = b" " * n
        err, = nvrtc.nvrtcGetPTX(prog, ptx)
        assert err == nvrtc.nvrtcResult.NVRTC_SUCCESS, err
        err, self.module = driver.cuModuleLoadData(ptx)
        assert err == driver.CUresult.CUDA_SUCCESS, err
        err, self.func = driver.cuModuleGetFunction(self.module, b"busy_rows")
        assert err == driver.CUresult.CUDA_SUCCESS, err
        self.rows, self.row_u4 = rows, row_bytes // 16
        gen = torch.Generator(device=device).manual_seed(11)
        self.src = torch.rand(rows * row_bytes // 4, device=device, generator=gen)   # finite positive floats
        self.sink = torch.zeros(1, device=device)
        self.stream = torch.cuda.Stream(device=device)

    def launch(self, times=1, blocks=148 * 8, reps=8):
        """Enqueue `times` launches on this object's stream, ordered after what the current stream holds now."""
        self.stream.wait_stream(torch.cuda.current_stream())
        args = ((self.src.data_ptr(), self.rows, self.row_u4, reps, self.sink.data_ptr()),
                (ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p))
        for _ in range(times):
            err, = self.driver.cuLaunchKernel(self.func, blocks, 1, 1, 128, 1, 1, 0, self.stream.cuda_stream, args, 0)
            assert err == self.driver.CUresult.CUDA_SUCCESS, err

    def close(self):
        torch.cuda.synchronize()
        self.driver.cuModuleUnload(self.module)
