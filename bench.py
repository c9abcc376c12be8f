#!/usr/bin/env python
"""Benchmark of the RAD training step on the wide bf16 MLP (8192 x 4 -> 1000, batch 65536).

A step is one pass of the whole hot path over one synthetic batch: for every layer the
Philox-masked compact store and the exact forward, then the loss, then per layer the weight
gradient from the store, the bias gradient and the exact input gradient.  The timed region
issues the per-layer C-ABI calls (the same launches rad_mlp_step makes) so CUDA events can
bracket each kernel family; the end-to-end figure goes through rad_mlp_step with the batch
coming from pinned host memory each step.

    python bench.py --gpus 1 --steps 5 --warmup 3
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N --master-addr 127.0.0.1 \
        --master-port P bench.py --gpus N --steps K --warmup W
    python bench.py --impl reference      # the CPU oracle on a row slab of the same workload

With N > 1 every rank runs an independent replica on its own batch (the path has no exchange
step: masks are keyed on global row indices and a real data-parallel job would only add one
all-reduce of dW); the reported value is all ranks' samples over the slowest rank's time.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "rad_train_step_samples_per_s"
SWEEP_PS = (0.01, 0.05, 0.1, 0.5)            # keep probabilities of the kernel sweep
UNIT = "samples/s"
DIMS = (8192, 8192, 8192, 8192, 8192, 1000)
BATCH = 65536
CPU_SLAB_ROWS = 2048         # rows of the workload the CPU oracle is timed on (10-30 s per step on 16 cores)
CPU_SLAB_ROWS_1CORE = 256    # rows for the single-core run of the same oracle (about the same wall time)
PHILOX_GCALLS_AT_MAX_CLOCK = 450.0   # Philox-4x32-10 calls per ns, register-only loop on one B200 at 1965 MHz


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--variant", default="different", choices=["different", "same", "project"])
    ap.add_argument("--law", default="bernoulli", choices=["bernoulli", "replace", "fixed"],
                    help="sampling law of the different / same variants")
    ap.add_argument("--p", type=float, default=0.1)
    ap.add_argument("--act", default="gelu", choices=["gelu", "relu"])
    ap.add_argument("--batch", type=int, default=BATCH)
    ap.add_argument("--no-sweep", action="store_true", help="skip the per-kernel p sweep")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    ap.add_argument("--no-twin", action="store_true", help="skip the timed ReLU twin of the wide net")
    ap.add_argument("--small-only", action="store_true",
                    help="run only the small workloads (MNIST-shaped MLP, IRNN, CNN) and print their figures")
    return ap.parse_args()


# --------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on a bounded row slab of the same workload
# --------------------------------------------------------------------------------------------
def _oracle_inputs(rows, seed=1234):
    from workloads import mlp_inputs
    return mlp_inputs(DIMS, rows, "bf16", "normal", seed)


def _blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


class _threads:
    """Limits the BLAS thread pool numpy uses (None: leave it alone)."""

    def __init__(self, n):
        self.n, self.ctx = n, None

    def __enter__(self):
        if self.n is not None:
            from threadpoolctl import threadpool_limits
            self.ctx = threadpool_limits(limits=self.n)
            self.ctx.__enter__()
        return self

    def __exit__(self, *exc):
        if self.ctx is not None:
            self.ctx.__exit__(*exc)


def time_oracle(args, steps, warmup, rows=CPU_SLAB_ROWS, threads=None):
    import numpy as np
    from oracle import rad as orc
    X, y, Ws, bs = _oracle_inputs(rows)
    times = []
    with _threads(threads):
        cores = _blas_threads() if threads is None else threads
        for i in range(warmup + steps):
            t0 = time.perf_counter()
            r = orc.mlp_step(X, y, Ws, bs, act=args.act, dtype="bf16", variant=args.variant, p=args.p, seed=0, step=i, law=args.law)
            dt = time.perf_counter() - t0
            if i >= warmup:
                times.append(dt)
            assert np.isfinite(r.loss)
    mean = sum(times) / len(times)
    return dict(value=rows / mean, unit=UNIT, cores=int(cores), kind="oracle",
                sample=f"row slab of {rows} rows of the same net (full D and H), "
                       f"{len(times)} step(s) of {mean:.2f} s"), mean


def time_small_oracles():
    """The oracle on the three small workloads at full size, all cores and one core (seconds per step)."""
    from oracle import rad as orc, irnn as oirnn, cnn as ocnn
    from workloads import cnn_inputs, irnn_inputs, mlp_inputs
    jobs = {}
    X, y, Ws, bs = mlp_inputs((784, 300, 300, 10), 150, "f32", "uniform01", 1234)
    jobs["mlp_784_300_300_10_b150_f32_different"] = (150, lambda: orc.mlp_step(X, y, Ws, bs, dtype="f32", variant="different", p=0.1, seed=0))
    jobs["mlp_784_300_300_10_b150_f32_same"] = (150, lambda: orc.mlp_step(X, y, Ws, bs, dtype="f32", variant="same", p=0.1, seed=0))
    ia = irnn_inputs(150, 784, 100, 10, 1234, True)
    jobs["irnn_h100_t784_b150_f32_different"] = (150, lambda: oirnn.irnn_step(*ia, variant="different", p=0.1, seed=0, step0=0))
    ca = cnn_inputs(128, 32, 3, (16, 32, 64), (128, 10), "bf16", 1234)
    jobs["cnn_32x32x3_c16_32_64_fc128_10_b128_bf16_different"] = (128, lambda: ocnn.cnn_step(*ca, dtype="bf16", variant="different", p=0.1, seed=0, step=0))
    out = {}
    for name, (batch, fn) in jobs.items():
        row = {}
        for label, threads in (("all_cores", None), ("one_core", 1)):
            with _threads(threads):
                fn()
                t0 = time.perf_counter()
                fn()
                dt = time.perf_counter() - t0
                row[label] = dict(samples_per_s=round(batch / dt, 1), s_per_step=round(dt, 4),
                                  cores=int(_blas_threads() if threads is None else threads))
        out[name] = row
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps, warmup = max(1, min(args.steps, 3)), min(args.warmup, 1)
    base, mean = time_oracle(args, steps, warmup)
    line = dict(impl="reference", metric=METRIC, value=base["value"], unit=UNIT, n_gpus=args.gpus, steps=steps,
                warmup=warmup, ms_per_step=mean * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic",
                config=dict(workload=f"mlp_wide: 8192->8192x4->1000 on the bf16 grid, batch {args.batch}; the oracle is "
                                     f"timed on a slab of {CPU_SLAB_ROWS} rows", dims=list(DIMS),
                            batch=CPU_SLAB_ROWS, variant=args.variant, law=args.law, p=args.p, act=args.act),
                cpu_baseline=base,
                e2e=dict(value=base["value"], unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------
def max_over_ranks(ms, device="cpu"):
    """Slowest rank's time: every rank contributes its own device time, all get the maximum."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world, batch_per_rank, steps, ms_total):
    """Samples per second of the whole job: all ranks' samples over the slowest rank's time."""
    return world * batch_per_rank * steps / (ms_total / 1e3)


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), power_w_max=max(power), samples=len(sm),
                    reasons=sorted(reasons))


class NvmlClock:
    """Current SM clock read through NVML (a read only; nothing is set)."""

    def __init__(self, index):
        self.h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv, self.h = pynvml, pynvml.nvmlDeviceGetHandleByIndex(index)
        except Exception:
            self.h = None

    def mhz(self):
        if self.h is None:
            return None
        try:
            return int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
        except Exception:
            return None


class LayerwiseStep:
    """The launches of rad_mlp_step issued call by call, with CUDA events around each kernel family."""

    def __init__(self, rad, torch, dims, B, act, variant, p, law="bernoulli"):
        self.rad, self.torch, self.dims, self.B, self.act, self.variant, self.p = rad, torch, dims, B, act, variant, p
        self.law = law
        L = self.L = len(dims) - 1
        dev, bf = "cuda", torch.bfloat16
        self.stores = [rad.Store(variant, "bf16", B, dims[l], p, layer=l, relu_bits=False, law=law) for l in range(L)]
        hid = max(dims[1:L]) if L > 1 else 8
        self.acts = [torch.empty(B, hid, dtype=bf, device=dev) for _ in range(2)]
        self.dzs = [torch.empty(B, max(dims[1:]), dtype=bf, device=dev) for _ in range(2)]
        self.logits = torch.empty(B, dims[L], dtype=torch.float32, device=dev)
        self.relubits = [None] + [torch.empty(B * ((dims[l] + 31) // 32), dtype=torch.int32, device=dev)
                                  if act == "relu" else None for l in range(1, L)]
        self.preact = [None] + [torch.empty(B, dims[l], dtype=bf, device=dev) if act == "gelu" else None
                                for l in range(1, L)]
        self.dW = [torch.empty(dims[l], dims[l + 1], dtype=torch.float32, device=dev) for l in range(L)]
        self.db = [torch.empty(dims[l + 1], dtype=torch.float32, device=dev) for l in range(L)]
        self.loss = torch.zeros(1, dtype=torch.float32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        ws = max([rad.rad_weight_grad_workspace(self.stores[l], dims[l + 1]) for l in range(L)] +
                 [rad.rad_input_grad_workspace(B, dims[l + 1]) for l in range(L)] + [B * 4, 256])
        self.ws = torch.empty(ws, dtype=torch.uint8, device=dev)
        self.events = []          # (family, layer, start, stop)

    def _timed(self, family, layer, fn):
        e0, e1 = self.torch.cuda.Event(enable_timing=True), self.torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        self.events.append((family, layer, e0, e1))

    def __call__(self, X, labels, Ws, bs, seed, step, record):
        rad, L, dims = self.rad, self.L, self.dims
        run = self._timed if record else (lambda fam, l, fn: fn())
        a_in = X
        # different-sample Bernoulli stores of hidden layers come out of the producing GEMM's epilogue; their
        # index part (key only) is timed with the store family, the GEMM with the forward family
        fused = self.variant == "different" and self.law in ("bernoulli", "fixed")
        for l in range(L):
            self.stores[l].c.seed, self.stores[l].c.step = seed, step
        st0 = self.stores[0]
        run("store", 0, lambda: rad.rad_linear_forward_store(a_in, st0, self.status))
        for l in range(L):
            last = l == L - 1
            if last:
                run("forward", l, lambda: rad.rad_linear_forward(a_in, Ws[l], bs[l], "none", out_z=self.logits,
                                                                 dev_status=self.status))
                break
            out = self.acts[l & 1][:, :dims[l + 1]]
            nxt = self.stores[l + 1]
            if self.variant == "redrawn":
                # the index part goes to the store's workspace inside the call and is not held
                run("forward", l, lambda: rad.rad_linear_forward_fill(a_in, Ws[l], bs[l], self.act, out, nxt,
                                                                      out_zlow=self.preact[l + 1],
                                                                      relubits=self.relubits[l + 1],
                                                                      dev_status=self.status))
            elif fused:
                run("store", l + 1, lambda: rad.rad_store_index(nxt, self.status))
                run("forward", l, lambda: rad.rad_linear_forward_fill(a_in, Ws[l], bs[l], self.act, out, nxt,
                                                                      out_zlow=self.preact[l + 1],
                                                                      relubits=self.relubits[l + 1], index_ready=True,
                                                                      dev_status=self.status))
            else:
                run("forward", l, lambda: rad.rad_linear_forward(a_in, Ws[l], bs[l], self.act, out_act=out,
                                                                 out_zlow=self.preact[l + 1],
                                                                 relubits=self.relubits[l + 1],
                                                                 dev_status=self.status))
                run("store", l + 1, lambda: rad.rad_linear_forward_store(out, nxt, self.status))
            a_in = out
        dz = self.dzs[(L - 1) & 1][:, :dims[L]]
        run("loss", L - 1, lambda: rad.rad_softmax_xent(self.logits, labels, self.loss, dz, self.ws))
        for l in range(L - 1, -1, -1):
            st = self.stores[l]
            run("dW", l, lambda: rad.rad_linear_weight_grad(st, dz, self.dW[l], self.ws, self.status))
            dz_prev = self.dzs[(l - 1) & 1][:, :dims[l]] if l > 0 else None
            # the call a user makes does both; here the column sums (db) and the GEMM are two calls, the same
            # launches in the same order, so that the GEMM's time is its own
            run("db", l, lambda: rad.rad_linear_input_grad(dz, Ws[l], db=self.db[l], workspace=self.ws, dev_status=self.status))
            if dz_prev is not None:
                run("dX", l, lambda: rad.rad_linear_input_grad(dz, Ws[l], relubits_prev=self.relubits[l],
                                                               z_prev=self.preact[l], dZ_prev=dz_prev,
                                                               workspace=self.ws, dev_status=self.status))
            dz = dz_prev

    def family_ms(self):
        out = {}
        for fam, layer, e0, e1 in self.events:
            out.setdefault((fam, layer), []).append(e0.elapsed_time(e1))
        return out


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=d["hbm_gbs"], tflops_burst=d["bf16_tflops"], tflops_sustained=d["bf16_tflops_sustained"],
                    sm_max_mhz=d.get("sm_max_mhz", 1965.0), source="measured")
    return dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, sm_max_mhz=1965.0, source="fallback")


def timed_alone(torch, fn, clock, n=10, settle_ms=60.0, idle_ms=0.0):
    """Median device time of `fn` timed alone (CUDA events on the launching stream) and the median SM clock
    read while the timed launches run.  `fn` first runs for about settle_ms so that the clock is the one
    this kernel sustains by itself, not what the kernels before it left behind.  idle_ms > 0: the device then
    rests that long and the timed launches are a burst after one more untimed launch (what a burst peak is
    compared with: the power cap answers within tens of milliseconds to the contractions before it)."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fn()
    torch.cuda.synchronize()
    e0.record(); fn(); e1.record()
    torch.cuda.synchronize()
    once = max(e0.elapsed_time(e1), 1e-3)
    for _ in range(max(2, min(400, int(settle_ms / once)))):
        fn()
    if idle_ms > 0.0:
        torch.cuda.synchronize()
        time.sleep(idle_ms / 1e3)
        fn()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
    ev[0].record()
    for i in range(n):
        fn()
        ev[i + 1].record()
    mhz = []
    while not ev[n].query():
        m = clock.mhz()
        if m is not None:
            mhz.append(m)
        time.sleep(0.0005)
    torch.cuda.synchronize()
    ms = statistics.median(ev[i].elapsed_time(ev[i + 1]) for i in range(n))
    return ms, (statistics.median(mhz) if mhz else None)


def store_bytes_different(B, D, nnz_padded, n_offsets, extra=0):
    """Algorithmic bytes of a different-sample store: the input read once, kept values (padded per tile),
    one keep bit per entry plus the row offsets that travel with them, one offset per tile."""
    ntiles = n_offsets - 1
    return B * D * 2 + nnz_padded * 2 + ntiles * 288 * 4 + 4 * n_offsets + extra


def sweep_stores(rad, torch, A, ps, clock):
    """The store kernels of the sweep, each timed alone.  Run before the timed steps: these kernels follow the SM
    clock, and after a minute of contractions at the power cap the part no longer gives its full clock even to a
    kernel that runs by itself (the clock read during the launches is reported beside every time)."""
    B, D = A.shape
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stores = {}
    for variant in ("different", "same"):
        for p in ps:
            st = rad.Store(variant, "bf16", B, D, p, relu_bits=False)
            ms_store, mhz = timed_alone(torch, lambda: rad.rad_linear_forward_store(A, st, status), clock, n=20, settle_ms=150.0)
            idx_t = None
            if variant == "different":
                idx_t = timed_alone(torch, lambda: rad.rad_store_index(st, status), clock, n=20, settle_ms=100.0)
            stores[(variant, p)] = (st, ms_store, mhz, idx_t)
    # the other sampling laws at fraction 0.1, and the static-shape form of the fixed-count law
    for law, variant in (("replace", "different"), ("replace", "same"), ("fixed", "different"), ("fixed", "same"), ("fixed", "rows")):
        st = rad.Store(variant, "bf16", B, D, 0.1, relu_bits=False, law=law)
        ms_store, mhz = timed_alone(torch, lambda: rad.rad_linear_forward_store(A, st, status), clock, n=10, settle_ms=100.0)
        stores[(variant, law)] = (st, ms_store, mhz, None)
    assert status.item() == 0, f"device status {status.item()}"
    return stores


def kernel_sweep(rad, torch, A, dZ, H, ps, pk, clock, stores):
    """Store and dW of one 8192 x 8192 layer, each kernel timed alone, for both variants over the p sweep (`stores`:
    what sweep_stores left; the weight gradients are timed here, from those stores)."""
    import numpy as np
    B, D = A.shape
    rows = []
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dW = torch.empty(D, H, dtype=torch.float32, device="cuda")
    hbm, burst = pk["hbm_gbs"], pk["tflops_burst"]

    def frac(v, peak):
        return round(v / peak, 4)

    for variant in ("different", "same"):
        for p in ps:
            st, ms_store, mhz, idx_t = stores.pop((variant, p))
            nnz = st.nnz.cpu().numpy()
            ws = torch.empty(max(rad.rad_weight_grad_workspace(st, H), 256), dtype=torch.uint8, device="cuda")
            ms_dw, mhz_dw = timed_alone(torch, lambda: rad.rad_linear_weight_grad(st, dZ, dW, ws, status), clock, n=5,
                                        settle_ms=30.0, idle_ms=150.0)
            row = dict(variant=variant, p=p, p_eff=rad.rad_effective_p(p), nnz=int(nnz[0]), store_ms=round(ms_store, 4),
                       store_sm_mhz=mhz, store_ms_x_mhz=None if mhz is None else round(ms_store * mhz, 1),
                       dW_ms=round(ms_dw, 4), dW_sm_mhz=mhz_dw)
            if variant == "different":
                sb = store_bytes_different(B, D, int(nnz[1]), len(st.offsets))
                row.update(store_bytes=sb, store_gbs=round(sb / ms_store / 1e6, 1), store_frac_hbm=frac(sb / ms_store / 1e6, hbm))
                ms_idx, mhz_idx = idx_t
                calls = 3.0 * B * D / 32
                row.update(index_ms=round(ms_idx, 4), index_sm_mhz=mhz_idx, index_philox_gcalls_s=round(calls / ms_idx / 1e6, 1))
                dense = 2.0 * B * D * H
                row.update(dW_tflops_dense_tile=round(dense / ms_dw / 1e9, 1), dW_frac_burst=frac(dense / ms_dw / 1e9, burst),
                           dW_useful_tflops=round(2.0 * int(nnz[0]) * H / ms_dw / 1e9, 1))
            else:
                k = int(nnz[0])
                idx = st.offsets[:k].cpu().numpy().view(np.uint32)
                sectors = int(np.unique(idx // 16).size)          # 32-byte sectors of a row that hold a kept column
                touched = B * sectors * 32 + B * int(st.c.values_ld) * 2 + 4 * k
                full = B * D * 2 + B * k * 2 + 4 * k
                row.update(store_bytes_touched=touched, store_gbs=round(touched / ms_store / 1e6, 1),
                           store_frac_hbm=frac(touched / ms_store / 1e6, hbm),
                           store_gbs_if_all_of_A_were_read=round(full / ms_store / 1e6, 1))
                flops = 2.0 * B * k * H
                # what this contraction has to move whatever p is: dZ once, the gathered block, dW written once
                dw_bytes = B * H * 2 + B * int(st.c.values_ld) * 2 + D * H * 4
                row.update(dW_tflops_kept_columns=round(flops / ms_dw / 1e9, 1), dW_frac_burst=frac(flops / ms_dw / 1e9, burst),
                           dW_bytes=dw_bytes, dW_gbs=round(dw_bytes / ms_dw / 1e6, 1), dW_frac_hbm=frac(dw_bytes / ms_dw / 1e6, hbm),
                           dW_bound="hbm" if dw_bytes / hbm / 1e6 > flops / burst / 1e9 else "tensor")
            rows.append(row)
            del st, ws
    # the paper's own law (k = ceil(fraction D) draws with replacement) and the fixed-count law without
    # replacement: index from the key alone + fill, then the same weight-gradient kernels on the store it leaves
    for law, variant in (("replace", "different"), ("replace", "same"), ("fixed", "different"), ("fixed", "same")):
        p = 0.1
        st, ms_store, mhz, _ = stores.pop((variant, law))
        nnz = st.nnz.cpu().numpy()
        ws = torch.empty(max(rad.rad_weight_grad_workspace(st, H), 256), dtype=torch.uint8, device="cuda")
        ms_dw, _ = timed_alone(torch, lambda: rad.rad_linear_weight_grad(st, dZ, dW, ws, status), clock, n=3, settle_ms=20.0, idle_ms=150.0)
        row = dict(variant=variant, law=law, p=p, draws_per_row=rad.rad_draws_per_row(p, D), nnz=int(nnz[0]),
                   store_ms=round(ms_store, 4), store_sm_mhz=mhz, dW_ms=round(ms_dw, 4))
        if variant == "different":
            # both laws make their index from the key alone: the algorithmic bytes are those of any bitmask store
            sb = store_bytes_different(B, D, int(nnz[1]), len(st.offsets))
            row.update(store_bytes=sb, store_gbs=round(sb / ms_store / 1e6, 1), store_frac_hbm=frac(sb / ms_store / 1e6, hbm),
                       held_bytes=int(nnz[1]) * 2 + (len(st.keepbits) + len(st.offsets)) * 4,
                       dW_tflops_dense_tile=round(2.0 * B * D * H / ms_dw / 1e9, 1),
                       dW_useful_tflops=round(2.0 * int(nnz[0]) * H / ms_dw / 1e9, 1))
        else:
            row.update(dW_tflops_kept_columns=round(2.0 * B * int(nnz[0]) * H / ms_dw / 1e9, 1))
        rows.append(row)
        del st, ws
    # the same-sample contraction against the kept-column count (fixed-count law: the count is exact): its time
    # follows the number of 256-column tiles, not their width
    for k in (416, 512, 768, 832, 1024, 2048):
        st = rad.Store("same", "bf16", B, D, k / D, relu_bits=False, law="fixed")
        rad.rad_linear_forward_store(A, st, status)
        ws = torch.empty(max(rad.rad_weight_grad_workspace(st, H), 256), dtype=torch.uint8, device="cuda")
        ms_dw, mhz_dw = timed_alone(torch, lambda: rad.rad_linear_weight_grad(st, dZ, dW, ws, status), clock, n=5, settle_ms=20.0,
                                    idle_ms=150.0)
        kk = int(st.nnz.cpu().numpy()[0])
        tf = 2.0 * B * kk * H / ms_dw / 1e9
        rows.append(dict(variant="same", law="fixed", kept_columns=kk, tiles=-(-kk // 256), dW_ms=round(ms_dw, 4), dW_sm_mhz=mhz_dw,
                         dW_tflops_kept_columns=round(tf, 1), dW_frac_burst=frac(tf, burst)))
        del st, ws
    # the fixed-count law in its static-shape form: B x k values and B x k 16-bit column numbers (k the same for
    # every row); the weight gradient rebuilds the tile-major index from the key and moves the values into it
    p = 0.1
    st, ms_store, mhz, _ = stores.pop(("rows", "fixed"))
    ws = torch.empty(max(rad.rad_weight_grad_workspace(st, H), 256), dtype=torch.uint8, device="cuda")
    ms_dw, _ = timed_alone(torch, lambda: rad.rad_linear_weight_grad(st, dZ, dW, ws, status), clock, n=3, settle_ms=20.0, idle_ms=150.0)
    k, ld = rad.rad_draws_per_row(p, D), int(st.c.values_ld)
    # bytes: the 32-byte sectors of A that hold a kept column (about 1 - (1 - k/D)^16 of them), values and columns written
    touched = int(B * D * 2 * (1.0 - (1.0 - k / D) ** 16)) + B * ld * 4
    rows.append(dict(variant="rows", law="fixed", p=p, kept_per_row=k, store_ms=round(ms_store, 4), store_sm_mhz=mhz,
                     store_bytes_touched=touched, store_gbs=round(touched / ms_store / 1e6, 1),
                     store_frac_hbm=frac(touched / ms_store / 1e6, hbm), held_bytes=B * ld * 4,
                     dW_ms=round(ms_dw, 4), dW_tflops_dense_tile=round(2.0 * B * D * H / ms_dw / 1e9, 1),
                     dW_useful_tflops=round(2.0 * B * k * H / ms_dw / 1e9, 1)))
    del st, ws
    # random projection (P = R R^T, Rademacher signs, k = ceil(0.1 D) columns): the store is one dense GEMM,
    # the weight gradient two; TFLOP/s on the flops of those contractions (2 B D k; 2 B k H + 2 D k H)
    p = 0.1
    st = rad.Store("project", "bf16", B, D, p, relu_bits=False)
    k = rad.rad_draws_per_row(p, D)
    ms_store, _ = timed_alone(torch, lambda: rad.rad_linear_forward_store(A, st, status), clock, n=5, settle_ms=20.0)
    ws = torch.empty(max(rad.rad_weight_grad_workspace(st, H), 256), dtype=torch.uint8, device="cuda")
    ms_dw, _ = timed_alone(torch, lambda: rad.rad_linear_weight_grad(st, dZ, dW, ws, status), clock, n=3, settle_ms=20.0, idle_ms=150.0)
    rows.append(dict(variant="project", p=p, k=k, store_ms=round(ms_store, 4),
                     store_tflops=round(2.0 * B * D * k / ms_store / 1e9, 1), dW_ms=round(ms_dw, 4),
                     dW_tflops=round((2.0 * B * k * H + 2.0 * D * k * H) / ms_dw / 1e9, 1), dW_flops="projected",
                     stored_bytes=int(st.c.values_ld) * B * 2))
    del st, ws
    assert status.item() == 0, f"device status {status.item()}"
    return rows


def small_workloads(rad, torch):
    """Samples/s of the small workloads (launch-latency bound; no roofline claim) with the launches per step."""
    import numpy as np
    from workloads import cnn_inputs, irnn_inputs, mlp_inputs
    out = {}

    def rate(fn, batch, reps):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        l0 = rad.rad_launch_count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(reps):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        return dict(samples_per_s=round(batch / ms * 1e3, 1), ms_per_step=round(ms, 4),
                    gpu_launches=int((rad.rad_launch_count() - l0) // reps))

    def memory(ctx, r):
        st = ctx.stats
        r["reserved_bytes"] = st.value_bytes + st.index_bytes + st.relu_bytes + st.unsampled_bytes
        r["full_backprop_bytes"] = st.full_backprop_bytes

    X, y, Ws, bs = mlp_inputs((784, 300, 300, 10), 150, "f32", "uniform01", 1234)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    Xd, yd, Wd, bd = dev(X), dev(y), [dev(W) for W in Ws], [dev(b) for b in bs]
    for variant in ("different", "same"):
        ctx = rad.MLPStep((784, 300, 300, 10), 150, "f32", "relu", variant, 0.1)
        r = rate(lambda i=0: ctx(Xd, yd, Wd, bd, seed=0, step=i), 150, 50)
        memory(ctx, r)
        held = rad.rad_mlp_held_bytes(ctx, ctx.nnz.cpu().tolist())
        r["held_bytes"] = held.value_bytes + held.index_bytes + held.relu_bytes + held.unsampled_bytes
        assert ctx.dev_status.item() == 0
        out["mlp_784_300_300_10_b150_f32_" + variant] = r
    args = [dev(a) for a in irnn_inputs(150, 784, 100, 10, 1234, True)]
    ctx = rad.IRNNStep(150, 784, 100, 10, "different", 0.1)
    r = rate(lambda i=0: ctx(*args, seed=0, step0=784 * i), 150, 20)
    memory(ctx, r)
    assert ctx.dev_status.item() == 0
    out["irnn_h100_t784_b150_f32_different"] = r
    X, y, cW, cb, fW, fb = cnn_inputs(128, 32, 3, (16, 32, 64), (128, 10), "bf16", 1234)
    bf = lambda a: dev(a).to(torch.bfloat16)
    cargs = (bf(X), dev(y), [bf(w) for w in cW], [dev(b) for b in cb], [bf(w) for w in fW], [dev(b) for b in fb])
    ctx = rad.CNNStep(128, 32, 3, (16, 32, 64), (128, 10), "bf16", "different", 0.1)
    r = rate(lambda i=0: ctx(*cargs, seed=0, step=i), 128, 20)
    memory(ctx, r)
    assert ctx.dev_status.item() == 0
    out["cnn_32x32x3_c16_32_64_fc128_10_b128_bf16_different"] = r
    # the same net with the convolutions of blocks 2 and 3 on CUDA cores instead of tensor cores, and both at a
    # batch large enough to leave the launch-bound regime
    conv = {}
    for batch in (128, 4096):
        Xb, yb, _, _, _, _ = cnn_inputs(batch, 32, 3, (16, 32, 64), (128, 10), "bf16", 1234)
        bargs = (bf(Xb), dev(yb)) + cargs[2:]
        for kern in ("tensor", "simt"):
            prev = rad.rad_set_conv_kernel(kern)
            try:
                c2 = rad.CNNStep(batch, 32, 3, (16, 32, 64), (128, 10), "bf16", "different", 0.1)
                rr = rate(lambda i=0: c2(*bargs, seed=0, step=i), batch, 10)
                assert c2.dev_status.item() == 0
            finally:
                rad.rad_set_conv_kernel(prev)
            conv[f"b{batch}_{kern}"] = dict(ms_per_step=rr["ms_per_step"], samples_per_s=rr["samples_per_s"])
            del c2
    out["cnn_32x32x3_c16_32_64_fc128_10_b128_bf16_different"]["conv_kernels"] = conv
    return out


def memory_report(rad, dims, B, act, variant, p, law, nnz_host):
    """Bytes held between the passes: as kept by the step that left `nnz_host`, and as reserved beforehand."""
    _, reserved = rad.rad_mlp_workspace(dims, B, "bf16", act, variant, p, law)
    held = rad.rad_mlp_held_bytes((dims, B, "bf16", act, variant, p, law), nnz_host)
    total = held.value_bytes + held.index_bytes + held.relu_bytes + held.preact_bytes + held.unsampled_bytes
    return dict(value_bytes=held.value_bytes, value_bytes_reserved=reserved.value_bytes, index_bytes=held.index_bytes,
                relu_bytes=held.relu_bytes, preact_bytes=held.preact_bytes, unsampled_bytes=held.unsampled_bytes,
                held_bytes=total, held_bytes_if_the_mask_is_redrawn_from_the_key=total - held.index_bytes,
                full_backprop_bytes=held.full_backprop_bytes, ratio=round(held.full_backprop_bytes / total, 3),
                ratio_if_the_mask_is_redrawn=round(held.full_backprop_bytes / (total - held.index_bytes), 3))


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2007_10412_b200 as rad

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B, dims, L = args.batch, DIMS, len(DIMS) - 1
    bf = torch.bfloat16
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1234 + rank)                       # every rank its own batch (weak scaling)
    X = torch.randn(B, dims[0], generator=gen, device="cuda", dtype=torch.float32).to(bf)
    labels = torch.randint(0, dims[L], (B,), generator=gen, device="cuda", dtype=torch.int32)
    wgen = torch.Generator(device="cuda")
    wgen.manual_seed(99)                               # same weights on every rank
    Ws = [(torch.randn(dims[l], dims[l + 1], generator=wgen, device="cuda") * (2.0 / dims[l]) ** 0.5).to(bf)
          for l in range(L)]
    bs = [torch.zeros(dims[l + 1], device="cuda") for l in range(L)]
    pk = peaks()
    clock = NvmlClock(local)
    # the store kernels of the sweep go first, while the part still gives a kernel that runs alone its full clock
    pre_stores = None
    if rank == 0 and world == 1 and not args.no_sweep:
        pre_stores = sweep_stores(rad, torch, X, SWEEP_PS, clock)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed_steps(lw, warmup, steps, first_step=0):
        for i in range(warmup):
            lw(X, labels, Ws, bs, seed=0, step=first_step + i, record=False)
        barrier()
        sampler = ClockSampler(local)
        sampler.start()
        launches0 = rad.rad_launch_count()
        t_start, t_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_start.record()
        for i in range(steps):
            lw(X, labels, Ws, bs, seed=0, step=first_step + warmup + i, record=True)
        t_stop.record()
        barrier()
        launches = (rad.rad_launch_count() - launches0) // max(steps, 1)
        clocks = sampler.stop()
        ms_total = max_over_ranks(t_start.elapsed_time(t_stop), "cuda")
        assert lw.status.item() == 0, f"device status {lw.status.item()}"
        return ms_total, launches, clocks

    lw = LayerwiseStep(rad, torch, dims, B, args.act, args.variant, args.p, args.law)
    ms_total, launches, clocks = timed_steps(lw, args.warmup, args.steps)
    ms_step = ms_total / args.steps
    value = whole_job_value(world, B, args.steps, ms_total)

    # per-family and per-kernel device time inside the timed region
    fam = lw.family_ms()
    by_family = {}
    for (f, l), v in fam.items():
        by_family.setdefault(f, 0.0)
        by_family[f] += sum(v) / args.steps

    def mean_ms(family, pick):
        t = [sum(v) / len(v) for (f, l), v in fam.items() if f == family and pick(l)]
        return sum(t) / len(t) if t else None

    big = lambda l: dims[l] == 8192 and dims[l + 1] == 8192
    fused = args.variant == "different" and args.law in ("bernoulli", "fixed")
    ms_fwd, ms_dw, ms_dx = mean_ms("forward", big), mean_ms("dW", big), mean_ms("dX", lambda l: big(l) and l > 0)
    ms_store0 = mean_ms("store", lambda l: l == 0)
    ms_store_hidden = mean_ms("store", lambda l: l > 0)      # fused: the key-only index kernels; else full stores
    nnz0 = lw.stores[0].nnz.cpu().numpy()
    nnz1 = lw.stores[1].nnz.cpu().numpy()
    dense = 2.0 * B * 8192 * 8192
    sust, burst, hbm = pk["tflops_sustained"], pk["tflops_burst"], pk["hbm_gbs"]

    def tensor_entry(what, ms, flops, extra=None):
        d = dict(kernel=what, bound="tensor", ms_per_launch=round(ms, 4), achieved=round(flops / ms / 1e9, 1), unit="TFLOP/s",
                 peak=sust, frac=round(flops / ms / 1e9 / sust, 4), peak_kind="sustained (kernel timed inside the step)")
        if extra:
            d.update(extra)
        return d

    kernels = {}
    kernels["forward"] = tensor_entry("tc_gemm_pair_kernel forward" + (" + next layer's store from the epilogue" if fused else ""),
                                      ms_fwd, dense)
    kernels["dX"] = tensor_entry("tc_gemm_pair_kernel input gradient", ms_dx, dense)
    if args.variant == "different":
        kernels["dW"] = tensor_entry("tc_sparse_pair_kernel, dense-tile flops 2*B*D*H", ms_dw, dense,
                                     dict(useful_tflops=round(2.0 * int(nnz1[0]) * 8192 / ms_dw / 1e9, 1)))
        sb = store_bytes_different(B, 8192, int(nnz0[1]), len(lw.stores[0].offsets),
                                   extra=2 * B * 8192 if args.law != "bernoulli" else 0)
        kernels["store"] = dict(kernel="store of the network input (stand-alone kernel)", bound="hbm", ms_per_launch=round(ms_store0, 4),
                                achieved=round(sb / ms_store0 / 1e6, 1), unit="GB/s", peak=hbm, frac=round(sb / ms_store0 / 1e6 / hbm, 4),
                                algorithmic_bytes=sb)
        if fused and args.law == "bernoulli":
            calls = 3.0 * B * 8192 / 32
            mhz = clocks.get("sm_mhz") or pk["sm_max_mhz"]
            peak_calls = PHILOX_GCALLS_AT_MAX_CLOCK * mhz / pk["sm_max_mhz"]
            kernels["store_index"] = dict(kernel="store_index_kernel + offsets_scan_kernel (hidden layers: index from the key, "
                                                 "values from the producing GEMM's epilogue)", bound="alu",
                                          ms_per_launch=round(ms_store_hidden, 4), achieved=round(calls / ms_store_hidden / 1e6, 1),
                                          unit="Philox Gcalls/s", peak=round(peak_calls, 1),
                                          frac=round(calls / ms_store_hidden / 1e6 / peak_calls, 4),
                                          peak_kind="register-only Philox loop, 450 Gcalls/s at 1965 MHz, scaled to the step's clock")
    elif args.variant == "same":
        k = int(nnz1[0])
        kernels["dW"] = tensor_entry("tc_gemm_pair_kernel same-sample dW (dW^T tile, kept columns on N), flops 2*B*k'*H", ms_dw,
                                     2.0 * B * k * 8192, dict(kept_columns=k))
        idx = lw.stores[0].offsets[:int(nnz0[0])].cpu().numpy()
        import numpy as np
        sectors = int(np.unique(idx.view(np.uint32) // 16).size)
        touched = B * sectors * 32 + B * int(lw.stores[0].c.values_ld) * 2
        kernels["store"] = dict(kernel="same-sample gather (bytes of the sectors it touches + the block written)", bound="hbm",
                                ms_per_launch=round(ms_store0, 4), achieved=round(touched / ms_store0 / 1e6, 1), unit="GB/s",
                                peak=hbm, frac=round(touched / ms_store0 / 1e6 / hbm, 4), algorithmic_bytes=touched)
    else:
        k = int(nnz1[0])
        kernels["dW"] = tensor_entry("projection dW: S^T dZ and R' G, flops 2*B*k*H + 2*D*k*H", ms_dw,
                                     2.0 * B * k * 8192 + 2.0 * 8192 * k * 8192)
        kernels["store"] = tensor_entry("projection store S = A R', flops 2*B*D*k", ms_store0, 2.0 * B * 8192 * k)
    dominant = max(("forward", "dW", "dX"), key=lambda f: by_family.get(f, 0.0))
    dom = kernels[dominant]
    # DRAM bytes per launch from the ncu captures under profiles/ (8192 x 8192 layer).  Two captures: one pass of
    # dram__bytes_read.sum + dram__bytes_write.sum over this very command at batch 65536, and the full set at batch
    # 8192; bytes read grow a little faster than the batch (the panels of a wave fall out of L2 sooner), so the
    # full-size figure serves from batch 32768 up and the small one, scaled by B / 8192, below.  The dW output does
    # not grow with the batch.  Only the default workload has a capture.
    traffic = None
    if args.act == "gelu" and abs(args.p - 0.1) < 1e-9 and args.law == "bernoulli" and args.variant == "different":
        big = B >= 32768
        if dominant == "forward":
            traffic = int((15.37e9 + 2.25e9) * B / 65536) if big else int((1263.5e6 + 269.8e6) * B / 8192)
        elif dominant == "dW":
            traffic = int(5.27e9 * B / 65536 + 0.25e9) if big else int(631.7e6 * B / 8192 + 236.0e6)
        elif dominant == "dX":
            traffic = int((17.68e9 + 1.07e9) * B / 65536) if big else None
    roofline = dict(bound=dom["bound"], kernel=dom["kernel"], achieved=dom["achieved"], peak=dom["peak"], unit=dom["unit"],
                    frac=dom["frac"], traffic=traffic, peak_source=pk["source"] + " (sustained cuBLAS bf16 / copy bandwidth)",
                    ms_per_launch=dom["ms_per_launch"],
                    how="CUDA events around each call on the launching stream, inside the timed steps",
                    kernels=kernels)

    # end to end through rad_mlp_step: the batch comes from pinned host memory every step
    ctx = rad.MLPStep(dims, B, "bf16", args.act, args.variant, args.p, law=args.law)
    Xh = torch.empty(X.shape, dtype=bf).pin_memory()
    Xh.copy_(X)
    yh = torch.empty(labels.shape, dtype=torch.int32).pin_memory()
    yh.copy_(labels)
    # Two device buffers: the copy of step i+1 runs on a copy stream under the kernels of step i, the
    # way an input pipeline feeds a trainer.  Every step's batch and labels are copied inside the
    # timed region (K copies, K steps), and every step's loss is read back to pinned host memory.
    Xd = [torch.empty_like(X) for _ in range(2)]
    yd = [torch.empty_like(labels) for _ in range(2)]
    del lw
    torch.cuda.empty_cache()
    copy_stream = torch.cuda.Stream()
    ready = [torch.cuda.Event() for _ in range(2)]
    freed = [torch.cuda.Event() for _ in range(2)]
    used = [False, False]
    loss_host = torch.zeros(max(args.steps, 2), dtype=torch.float32).pin_memory()

    def issue_copy(i):
        b = i & 1
        with torch.cuda.stream(copy_stream):
            if used[b]:
                copy_stream.wait_event(freed[b])
            Xd[b].copy_(Xh, non_blocking=True)
            yd[b].copy_(yh, non_blocking=True)
            ready[b].record(copy_stream)

    def issue_step(i, step_no):
        b = i & 1
        cur = torch.cuda.current_stream()
        cur.wait_event(ready[b])
        ctx(Xd[b], yd[b], Ws, bs, seed=0, step=step_no)
        freed[b].record(cur)
        used[b] = True
        loss_host[i:i + 1].copy_(ctx.loss.reshape(1), non_blocking=True)

    def e2e_run(n, first_step):
        issue_copy(0)
        for i in range(n):
            if i + 1 < n:
                issue_copy(i + 1)
            issue_step(i, first_step + i)

    e2e_run(min(args.warmup, 2), 0)
    torch.cuda.synchronize()
    barrier()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    e2e_run(args.steps, 100)
    e1.record()
    torch.cuda.synchronize()
    loss = float(loss_host[args.steps - 1])
    barrier()
    e2e_ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3 if world == 1 else 0.0)
    e2e_ms = max_over_ranks(e2e_ms, "cuda")
    assert ctx.dev_status.item() == 0
    e2e = dict(value=whole_job_value(world, B, args.steps, e2e_ms), unit=UNIT,
               h2d_bytes_per_step=Xh.numel() * 2 + yh.numel() * 4, d2h_bytes_per_step=4,
               ms_per_step=round(e2e_ms / args.steps, 3), api="rad_mlp_step", last_loss=round(loss, 5),
               pipeline="two device input buffers; the host-to-device copy of step i+1 runs on a copy stream "
                        "under step i; K copies and K steps inside the timed region")
    # stored activation bytes versus full backprop, from the counts the last step left
    memory = memory_report(rad, dims, B, args.act, args.variant, args.p, args.law, ctx.nnz.cpu().tolist())
    del ctx, Xd, yd
    torch.cuda.empty_cache()

    # The same shapes with ReLU: 1-bit derivatives instead of kept pre-activations, the setting of the
    # paper's memory figures (App. A).  Timed for real: one warm-up step, then `twin_steps` steps.
    twin = None
    if args.act != "relu" and rank == 0 and world == 1 and not args.no_twin:
        lw2 = LayerwiseStep(rad, torch, dims, B, "relu", args.variant, args.p, args.law)
        twin_steps = min(args.steps, 2)
        ms2, launches2, _ = timed_steps(lw2, 1, twin_steps, first_step=50)
        nnz_all = []
        for st in lw2.stores:
            nnz_all += st.nnz.cpu().tolist()
        twin = dict(act="relu", steps=twin_steps, ms_per_step=round(ms2 / twin_steps, 3),
                    samples_per_s=round(B * twin_steps / (ms2 / 1e3), 1), gpu_launches=int(launches2),
                    family_ms={k: round(sum(sum(v) for (f, l), v in lw2.family_ms().items() if f == k) / twin_steps, 3)
                               for k in ("store", "forward", "loss", "dW", "dX", "db")},
                    activation_memory=memory_report(rad, dims, B, "relu", args.variant, args.p, args.law, nnz_all))
        del lw2
        torch.cuda.empty_cache()
        if args.variant == "different" and args.law in ("bernoulli", "fixed"):
            # the same twin holding no keep bits: every index is drawn again from the key in the backward pass
            lw3 = LayerwiseStep(rad, torch, dims, B, "relu", "redrawn", args.p, args.law)
            ms3, launches3, _ = timed_steps(lw3, 1, twin_steps, first_step=60)
            nnz_all = []
            for st in lw3.stores:
                nnz_all += st.nnz.cpu().tolist()
            twin["mask_redrawn"] = dict(
                variant="redrawn", steps=twin_steps, ms_per_step=round(ms3 / twin_steps, 3),
                samples_per_s=round(B * twin_steps / (ms3 / 1e3), 1), gpu_launches=int(launches3),
                family_ms={k: round(sum(sum(v) for (f, l), v in lw3.family_ms().items() if f == k) / twin_steps, 3)
                           for k in ("store", "forward", "loss", "dW", "dX", "db")},
                activation_memory=memory_report(rad, dims, B, "relu", "redrawn", args.p, args.law, nnz_all))
            del lw3
            torch.cuda.empty_cache()

    sweep = None
    if rank == 0 and world == 1 and not args.no_sweep:
        dZ = (torch.randn(B, 8192, generator=gen, device="cuda") / B).to(bf)
        sweep = kernel_sweep(rad, torch, X, dZ, 8192, SWEEP_PS, pk, clock, pre_stores)
        # the two kernels the targets are set for, timed alone at this run's p, beside their in-step figures
        for row in sweep:
            if row.get("law") is None and row["variant"] == args.variant and abs(row["p"] - args.p) < 1e-9:
                if "store" in kernels and "store_frac_hbm" in row:
                    kernels["store"]["alone"] = dict(ms=row["store_ms"], achieved=row["store_gbs"], frac=row["store_frac_hbm"],
                                                     sm_mhz=row["store_sm_mhz"], peak=hbm, unit="GB/s")
                kernels["dW"]["alone"] = dict(ms=row["dW_ms"], achieved=row.get("dW_tflops_dense_tile", row.get("dW_tflops_kept_columns")),
                                              frac=row["dW_frac_burst"], peak=burst, unit="TFLOP/s", peak_kind="burst")
        del dZ
    small = small_workloads(rad, torch) if (rank == 0 and world == 1 and not args.no_sweep) else None
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu, _ = time_oracle(args, 1, 0)
        one, _ = time_oracle(args, 1, 0, rows=CPU_SLAB_ROWS_1CORE, threads=1)
        cpu["one_core"] = one
        if small is not None:
            for name, row in time_small_oracles().items():
                small[name]["cpu_oracle"] = row

    if rank == 0:
        pe = rad.rad_effective_p(args.p)
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                    ms_per_step=ms_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                    data="synthetic",
                    config=dict(workload=f"mlp_wide: 8192->8192x4->1000, bf16, batch {B} per GPU, N(0,1) inputs",
                                dims=list(dims), global_batch=world * B, act=args.act, variant=args.variant, law=args.law, p=args.p,
                                p_sampled=pe, parallelism="replicas" if world > 1 else "1 GPU",
                                l2="inputs larger than L2 (1 GiB activations per layer)", sm_pairs=rad.rad_sm_pairs()),
                    clocks=clocks, e2e=e2e, gpu_launches=int(launches), roofline=roofline,
                    family_ms={k: round(v, 3) for k, v in by_family.items()},
                    activation_memory=memory, relu_twin=twin, cpu_baseline=cpu, kernel_sweep=sweep, small_workloads=small)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_small_only():
    import torch
    import paper_2007_10412_b200 as rad
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    print(json.dumps(dict(small_workloads=small_workloads(rad, torch))))


def main():
    args = parse_args()
    if args.small_only:
        if int(os.environ.get("RANK", "0")) == 0:
            run_small_only()
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
