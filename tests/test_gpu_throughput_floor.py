"""Throughput floors: every kernel variant that serves a common shape must stay within reach of the memory
system.  The floors are loose (about 60 % of what this library measures on a B200, so that a shared or
power-capped board does not trip them) but a variant that falls off a cliff -- a register spill in a hot loop
once cost the static-slot bf16 kernel a factor 2.6 while every parity test stayed green -- fails here.
Timed with CUDA events on device-resident buffers, three rotating sets, best of five batches."""
import pytest
import torch

pytestmark = pytest.mark.gpu

ES = {torch.float32: 4, torch.bfloat16: 2, torch.complex64: 8}


def tb_per_s(hs, rows, n, dtype, call, offset=0, tune=()):
    cnt = rows * n
    g = torch.Generator(device="cuda").manual_seed(rows * 31 + n)

    def place(t):
        buf = torch.empty(cnt + 16, dtype=t.dtype, device="cuda")
        v = buf[offset:offset + cnt].view(rows, n)
        v.copy_(t)
        return v

    def real(scale, shift):
        return torch.randn(rows, n, device="cuda", generator=g) * scale + shift

    sets = []
    for _ in range(3):
        if dtype == torch.complex64:
            sign = lambda: (torch.rand(rows, n, device="cuda", generator=g) < 0.5).float() * torch.pi
            a, b = torch.complex(real(0.1, -0.3), sign()), torch.complex(real(1.0, 0.0), sign())
            x0 = torch.complex(torch.zeros(rows, device="cuda"), torch.zeros(rows, device="cuda"))
        elif call == "linear":
            a = (torch.rand(rows, n, device="cuda", generator=g) * 0.5 + 0.5) * torch.sign(real(1.0, 0.0))
            b, x0 = real(1.0, 0.0), torch.randn(rows, device="cuda", generator=g)
        else:
            a, b, x0 = real(0.05, -0.1).to(dtype), real(1.0, 0.0).to(dtype), torch.zeros(rows, dtype=dtype, device="cuda")
        a, b = place(a), place(b)
        out = torch.empty(cnt + 16, dtype=a.dtype, device="cuda")[offset:offset + cnt].view(rows, n)
        if dtype == torch.complex64:
            ws = torch.empty(int(hs.lib().heinsen_scan_complex_workspace_bytes(rows, n)), dtype=torch.uint8, device="cuda")
        else:
            ws = hs.new_workspace(rows, n, "cuda")
        sets.append((a, b, x0, out, ws))

    def step(i):
        a, b, x0, out, ws = sets[i % 3]
        if dtype == torch.complex64:
            hs.scan_log_complex(a, b, x0, log_x=out, workspace=ws)
        elif call == "linear":
            hs.scan_linear(a, b, x0, x=out, workspace=ws)
        else:
            hs.scan_log(a, b, x0, log_x=out, workspace=ws)

    for name, value in tune:
        hs.tune(name, value)
    try:
        for i in range(4):
            step(i)
        torch.cuda.synchronize()
        for s in sets:
            hs.check(s[4])
        best = float("inf")
        for _ in range(5):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(12):
                step(i)
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1) / 12)
    finally:
        for name, _ in tune:
            hs.tune(name, -1)
    return cnt * 3 * ES[dtype] / (best * 1e-3) / 1e12


@pytest.mark.parametrize("what,rows,n,dtype,call,offset,tune,floor", [
    ("fp32 log, tickets (configuration 2)", 16384, 2048, torch.float32, "log", 0, (), 3.8),
    ("fp32 log, static slots", 4096, 8192, torch.float32, "log", 0, (), 3.6),
    ("fp32 signed linear (configuration 4)", 4096, 8192, torch.float32, "linear", 0, (), 3.4),
    ("bf16 log, static slots", 4096, 16384, torch.bfloat16, "log", 0, (), 3.2),
    ("bf16 log, tickets", 16384, 4096, torch.bfloat16, "log", 0, (), 3.2),
    ("complex logarithms", 2048, 8192, torch.complex64, "log", 0, (), 3.2),
    ("fp32 short rows, several rows per warp", 262144, 128, torch.float32, "log", 0, (), 3.4),
    ("fp32 rows TMA cannot address", 16384, 2047, torch.float32, "log", 0, (), 3.0),
    ("fp32 rows from an odd base", 16384, 2048, torch.float32, "log", 1, (), 3.0),
    ("bf16 rows TMA cannot address", 16384, 2047, torch.bfloat16, "log", 0, (), 2.0),
    ("fp32 single sequence, look-back (configuration 3 at a quarter)", 1, 1 << 24, torch.float32, "log", 0, (), 2.4),
    ("fp32 linear single sequence, look-back", 1, 1 << 24, torch.float32, "linear", 0, (), 1.8),
])
def test_throughput_floor(hs, what, rows, n, dtype, call, offset, tune, floor):
    got = tb_per_s(hs, rows, n, dtype, call, offset, tune)
    assert got >= floor, f"{what}: {got:.2f} TB/s of algorithmic traffic, floor {floor} TB/s"
