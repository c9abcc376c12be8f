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
UNIT = "samples/s"
DIMS = (8192, 8192, 8192, 8192, 8192, 1000)
BATCH = 65536
CPU_SLAB_ROWS = 2048         # rows of the workload the CPU oracle is timed on (10-30 s per step on 16 cores)


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
    return ap.parse_args()


# --------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on a bounded row slab of the same workload
# --------------------------------------------------------------------------------------------
def _oracle_inputs(rows, seed=1234):
    from workloads import mlp_inputs
    return mlp_inputs(DIMS, rows, "bf16", "normal", seed)


def time_oracle(args, steps, warmup):
    import numpy as np
    from oracle import rad as orc
    try:
        from threadpoolctl import threadpool_info
        cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    X, y, Ws, bs = _oracle_inputs(CPU_SLAB_ROWS)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        r = orc.mlp_step(X, y, Ws, bs, act=args.act, dtype="bf16", variant=args.variant, p=args.p, seed=0, step=i, law=args.law)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
        assert np.isfinite(r.loss)
    mean = sum(times) / len(times)
    return dict(value=CPU_SLAB_ROWS / mean, unit=UNIT, cores=int(cores), kind="oracle",
                sample=f"row slab of {CPU_SLAB_ROWS} rows of the same net (full D and H), "
                       f"{len(times)} step(s) of {mean:.2f} s"), mean


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps, warmup = max(1, min(args.steps, 3)), min(args.warmup, 1)
    base, mean = time_oracle(args, steps, warmup)
    line = dict(impl="reference", metric=METRIC, value=base["value"], unit=UNIT, n_gpus=args.gpus, steps=steps,
                warmup=warmup, ms_per_step=mean * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic",
                config=dict(workload="mlp_wide 8192x4->1000 bf16 grid, oracle on a row slab", dims=list(DIMS),
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
        fused = self.variant == "different" and self.law == "bernoulli"
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
            if fused:
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
            run("dX+db", l, lambda: rad.rad_linear_input_grad(dz, Ws[l], relubits_prev=self.relubits[l],
                                                              z_prev=self.preact[l], dZ_prev=dz_prev, db=self.db[l],
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
                    source="measured")
    return dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, source="fallback")


def kernel_sweep(rad, torch, A, dZ, H, ps):
    """Store GB/s and dW TFLOP/s of one 8192 x 8192 layer for both variants over the p sweep."""
    B, D = A.shape
    rows = []
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dW = torch.empty(D, H, dtype=torch.float32, device="cuda")

    def timed(fn, n=5):
        fn(); fn()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
        ev[0].record()
        for i in range(n):
            fn()
            ev[i + 1].record()
        torch.cuda.synchronize()
        return statistics.median(ev[i].elapsed_time(ev[i + 1]) for i in range(n))

    for variant in ("different", "same"):
        for p in ps:
            st = rad.Store(variant, "bf16", B, D, p, relu_bits=False)
            ms_store = timed(lambda: rad.rad_linear_forward_store(A, st, status))
            nnz = st.nnz.cpu().numpy()
            ws = torch.empty(max(rad.rad_weight_grad_workspace(st, H), 256), dtype=torch.uint8, device="cuda")
            ms_dw = timed(lambda: rad.rad_linear_weight_grad(st, dZ, dW, ws, status), n=3)
            if variant == "different":
                store_bytes = B * D * 2 + int(nnz[1]) * 2 + B * D // 8 + 4 * (len(st.offsets))
                flops, kind = 2.0 * B * D * H, "dense-tile"
            else:
                store_bytes = B * D * 2 + int(nnz[1]) * 2 + 4 * int(nnz[0])
                flops, kind = 2.0 * B * int(nnz[0]) * H, "kept-columns"
            rows.append(dict(variant=variant, p=p, store_ms=round(ms_store, 4),
                             store_gbs=round(store_bytes / ms_store / 1e6, 1),
                             dW_ms=round(ms_dw, 4), dW_tflops=round(flops / ms_dw / 1e9, 1), dW_flops=kind,
                             nnz=int(nnz[0])))
            del st, ws
    # the paper's own law (k = ceil(fraction D) draws with replacement) and the fixed-count law without
    # replacement: multiplicity kernel + store, then the same weight-gradient kernels on the store it leaves
    for law, variant in (("replace", "different"), ("replace", "same"), ("fixed", "different"), ("fixed", "same")):
        p = 0.1
        st = rad.Store(variant, "bf16", B, D, p, relu_bits=False, law=law)
        ms_store = timed(lambda: rad.rad_linear_forward_store(A, st, status))
        nnz = st.nnz.cpu().numpy()
        ws = torch.empty(max(rad.rad_weight_grad_workspace(st, H), 256), dtype=torch.uint8, device="cuda")
        ms_dw = timed(lambda: rad.rad_linear_weight_grad(st, dZ, dW, ws, status), n=3)
        if variant == "different":
            # the multiplicity matrix (a byte per entry) is written and read once on top of the store's bytes
            store_bytes = B * D * 2 + int(nnz[1]) * 2 + B * D // 8 + 4 * len(st.offsets) + 2 * B * D
            flops, kind = 2.0 * B * D * H, "dense-tile"
        else:
            store_bytes = B * D * 2 + int(nnz[1]) * 2 + 4 * int(nnz[0])
            flops, kind = 2.0 * B * int(nnz[0]) * H, "kept-columns"
        rows.append(dict(variant=variant, law=law, p=p, draws_per_row=rad.rad_draws_per_row(p, D),
                         store_ms=round(ms_store, 4), store_gbs=round(store_bytes / ms_store / 1e6, 1),
                         dW_ms=round(ms_dw, 4), dW_tflops=round(flops / ms_dw / 1e9, 1), dW_flops=kind,
                         nnz=int(nnz[0])))
        del st, ws
    # random projection (P = R R^T, Rademacher signs, k = ceil(0.1 D) columns): the store is one dense GEMM,
    # the weight gradient two; TFLOP/s on the flops of those contractions (2 B D k; 2 B k H + 2 D k H)
    p = 0.1
    st = rad.Store("project", "bf16", B, D, p, relu_bits=False)
    k = rad.rad_draws_per_row(p, D)
    ms_store = timed(lambda: rad.rad_linear_forward_store(A, st, status))
    ws = torch.empty(max(rad.rad_weight_grad_workspace(st, H), 256), dtype=torch.uint8, device="cuda")
    ms_dw = timed(lambda: rad.rad_linear_weight_grad(st, dZ, dW, ws, status), n=3)
    rows.append(dict(variant="project", p=p, k=k, store_ms=round(ms_store, 4),
                     store_tflops=round(2.0 * B * D * k / ms_store / 1e9, 1), dW_ms=round(ms_dw, 4),
                     dW_tflops=round((2.0 * B * k * H + 2.0 * D * k * H) / ms_dw / 1e9, 1), dW_flops="projected",
                     stored_bytes=int(st.c.values_ld) * B * 2))
    del st, ws
    assert status.item() == 0, f"device status {status.item()}"
    return rows


def small_workloads(rad, torch):
    """Samples/s of the two small float32 workloads (launch-latency bound; no roofline claim)."""
    import numpy as np
    from workloads import irnn_inputs, mlp_inputs
    out = {}

    def rate(fn, batch, reps):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(reps):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        return dict(samples_per_s=round(batch / ms * 1e3, 1), ms_per_step=round(ms, 4))

    X, y, Ws, bs = mlp_inputs((784, 300, 300, 10), 150, "f32", "uniform01", 1234)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    Xd, yd, Wd, bd = dev(X), dev(y), [dev(W) for W in Ws], [dev(b) for b in bs]
    for variant in ("different", "same"):
        ctx = rad.MLPStep((784, 300, 300, 10), 150, "f32", "relu", variant, 0.1)
        r = rate(lambda i=0: ctx(Xd, yd, Wd, bd, seed=0, step=i), 150, 50)
        st = ctx.stats
        r["held_bytes"] = st.value_bytes + st.index_bytes + st.relu_bytes + st.unsampled_bytes
        r["full_backprop_bytes"] = st.full_backprop_bytes
        assert ctx.dev_status.item() == 0
        out["mlp_784_300_300_10_b150_f32_" + variant] = r
    args = [dev(a) for a in irnn_inputs(150, 784, 100, 10, 1234, True)]
    ctx = rad.IRNNStep(150, 784, 100, 10, "different", 0.1)
    r = rate(lambda i=0: ctx(*args, seed=0, step0=784 * i), 150, 20)
    st = ctx.stats
    r["held_bytes"] = st.value_bytes + st.index_bytes + st.relu_bytes + st.unsampled_bytes
    r["full_backprop_bytes"] = st.full_backprop_bytes
    assert ctx.dev_status.item() == 0
    out["irnn_h100_t784_b150_f32_different"] = r
    from workloads import cnn_inputs
    X, y, cW, cb, fW, fb = cnn_inputs(128, 32, 3, (16, 32, 64), (128, 10), "bf16", 1234)
    bf = lambda a: dev(a).to(torch.bfloat16)
    cargs = (bf(X), dev(y), [bf(w) for w in cW], [dev(b) for b in cb], [bf(w) for w in fW], [dev(b) for b in fb])
    ctx = rad.CNNStep(128, 32, 3, (16, 32, 64), (128, 10), "bf16", "different", 0.1)
    r = rate(lambda i=0: ctx(*cargs, seed=0, step=i), 128, 20)
    st = ctx.stats
    r["held_bytes"] = st.value_bytes + st.index_bytes + st.relu_bytes + st.unsampled_bytes
    r["full_backprop_bytes"] = st.full_backprop_bytes
    assert ctx.dev_status.item() == 0
    out["cnn_32x32x3_c16_32_64_fc128_10_b128_bf16_different"] = r
    return out


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

    lw = LayerwiseStep(rad, torch, dims, B, args.act, args.variant, args.p, args.law)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        lw(X, labels, Ws, bs, seed=0, step=i, record=False)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = rad.rad_launch_count()
    t_start, t_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(args.steps):
        lw(X, labels, Ws, bs, seed=0, step=args.warmup + i, record=True)
    t_stop.record()
    barrier()
    launches = (rad.rad_launch_count() - launches0) // max(args.steps, 1)
    clocks = sampler.stop()
    ms_total = t_start.elapsed_time(t_stop)
    ms_total = max_over_ranks(ms_total, "cuda")
    assert lw.status.item() == 0, f"device status {lw.status.item()}"
    ms_step = ms_total / args.steps
    value = whole_job_value(world, B, args.steps, ms_total)

    # per-family device time inside the timed region, and the roofline of the dominant kernel
    fam = lw.family_ms()
    by_family = {}
    for (f, l), v in fam.items():
        by_family.setdefault(f, 0.0)
        by_family[f] += sum(v) / args.steps
    pk = peaks()
    dw_big = [(l, sum(v) / len(v)) for (f, l), v in fam.items() if f == "dW" and dims[l] == 8192 and dims[l + 1] == 8192]
    fwd_big = [(l, sum(v) / len(v)) for (f, l), v in fam.items() if f == "forward" and dims[l + 1] == 8192]
    dominant = max(by_family, key=by_family.get)
    if dominant == "dW":
        ms_k = sum(t for _, t in dw_big) / len(dw_big)
        if args.variant == "different":
            flops, what = 2.0 * B * 8192 * 8192, "tc_sparse_pair_kernel (different-sample dW), dense-tile flops 2*B*D*H"
        elif args.variant == "project":
            k = int(lw.stores[1].nnz[0].item())
            flops, what = 2.0 * B * k * 8192 + 2.0 * 8192 * k * 8192, "projection dW: S^T dZ and R' G, flops 2*B*k*H + 2*D*k*H"
        else:
            k = int(lw.stores[1].nnz[0].item())
            flops, what = 2.0 * B * k * 8192, "tc_gemm_pair_kernel<MN,MN> (same-sample dW), flops 2*B*k'*H on kept columns"
    else:
        ms_k = sum(t for _, t in fwd_big) / len(fwd_big)
        flops, what = 2.0 * B * 8192 * 8192, "tc_gemm_pair_kernel forward, flops 2*B*D*H"
    achieved = flops / ms_k / 1e9
    # DRAM bytes per launch from the ncu captures under profiles/ (batch 8192, 8192 x 8192 layer): bytes
    # read grow with the batch and are scaled by B / 8192, the dW output does not grow.  Only the
    # default workload has a capture.
    traffic = None
    if args.act == "gelu" and abs(args.p - 0.1) < 1e-9 and args.law == "bernoulli":
        if dominant == "dW" and args.variant == "different":
            traffic = int(351.5e6 * B / 8192 + 228.4e6)
        elif dominant != "dW":
            traffic = int((1095.8e6 + 251.4e6) * B / 8192)
    roofline = dict(bound="tensor", kernel=what, achieved=round(achieved, 1), peak=pk["tflops_sustained"],
                    unit="TFLOP/s", frac=round(achieved / pk["tflops_sustained"], 4), traffic=traffic,
                    peak_source=pk["source"] + " (sustained cuBLAS bf16)", ms_per_launch=round(ms_k, 4),
                    how="CUDA events around the call on the launching stream, inside the timed steps")
    store_big = [sum(v) / len(v) for (f, l), v in fam.items() if f == "store" and dims[l] == 8192]
    nnz1 = lw.stores[1].nnz.cpu().numpy()
    if args.variant == "different":
        sbytes = B * 8192 * 2 + int(nnz1[1]) * 2 + B * 8192 // 8 + 4 * len(lw.stores[1].offsets)
        if args.law != "bernoulli":
            sbytes += 2 * B * 8192                     # the multiplicity matrix, written and read once
    else:
        sbytes = B * 8192 * 2 + int(nnz1[1]) * 2 + 4 * int(nnz1[0])
    ms_s = sum(store_big) / len(store_big)
    if args.variant == "project":
        # the store of this variant is a dense contraction (S = A R'), not a streaming kernel
        sflops = 2.0 * B * 8192 * int(nnz1[0])
        store_roofline = dict(bound="tensor", kernel="projection store S = A R', flops 2*B*D*k",
                              achieved=round(sflops / ms_s / 1e9, 1), peak=pk["tflops_sustained"], unit="TFLOP/s",
                              frac=round(sflops / ms_s / 1e9 / pk["tflops_sustained"], 4), traffic=None,
                              ms_per_launch=round(ms_s, 4))
    else:
        store_roofline = dict(bound="hbm", kernel="store kernel, one 8192-wide layer input",
                              achieved=round(sbytes / ms_s / 1e6, 1), peak=pk["hbm_gbs"], unit="GB/s",
                              frac=round(sbytes / ms_s / 1e6 / pk["hbm_gbs"], 4),
                              traffic=(int((134.3e6 + 16.2e6) * B / 8192)
                                       if args.variant == "different" and args.law == "bernoulli" and
                                       abs(args.p - 0.1) < 1e-9 else None),
                              ms_per_launch=round(ms_s, 4), algorithmic_bytes=sbytes)

    # stored activation bytes versus full backprop (from the whole-net entry point's plan)
    ctx = rad.MLPStep(dims, B, "bf16", args.act, args.variant, args.p, law=args.law)
    s = ctx.stats
    held = s.value_bytes + s.index_bytes + s.relu_bytes + s.preact_bytes + s.unsampled_bytes
    memory = dict(value_bytes=s.value_bytes, index_bytes=s.index_bytes, relu_bytes=s.relu_bytes,
                  preact_bytes=s.preact_bytes, unsampled_bytes=s.unsampled_bytes, held_bytes=held,
                  full_backprop_bytes=s.full_backprop_bytes, ratio=round(s.full_backprop_bytes / held, 3))

    # the same shapes with ReLU (1-bit derivatives instead of kept pre-activations): plan only, not run
    if args.act != "relu":
        _, sr = rad.rad_mlp_workspace(dims, B, "bf16", "relu", args.variant, args.p, args.law)
        held_r = sr.value_bytes + sr.index_bytes + sr.relu_bytes + sr.preact_bytes + sr.unsampled_bytes
        memory["same_shapes_relu"] = dict(value_bytes=sr.value_bytes, index_bytes=sr.index_bytes, relu_bytes=sr.relu_bytes,
                                          preact_bytes=sr.preact_bytes, unsampled_bytes=sr.unsampled_bytes,
                                          held_bytes=held_r, full_backprop_bytes=sr.full_backprop_bytes,
                                          ratio=round(sr.full_backprop_bytes / held_r, 3))

    # end to end through rad_mlp_step: the batch comes from pinned host memory every step
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

    sweep = None
    if rank == 0 and world == 1 and not args.no_sweep:
        dZ = (torch.randn(B, 8192, generator=gen, device="cuda") / B).to(bf)
        sweep = kernel_sweep(rad, torch, X, dZ, 8192, (0.01, 0.05, 0.1, 0.5))
    small = small_workloads(rad, torch) if (rank == 0 and world == 1 and not args.no_sweep) else None
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu, _ = time_oracle(args, 1, 0)

    if rank == 0:
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                    ms_per_step=ms_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                    data="synthetic",
                    config=dict(workload="mlp_wide: 8192->8192x4->1000, bf16, batch 65536 per GPU, N(0,1) inputs",
                                dims=list(dims), global_batch=world * B, act=args.act, variant=args.variant, law=args.law, p=args.p,
                                parallelism="replicas" if world > 1 else "1 GPU",
                                l2="inputs larger than L2 (1 GiB activations per layer)"),
                    clocks=clocks, e2e=e2e, gpu_launches=int(launches), roofline=roofline,
                    store_roofline=store_roofline, family_ms={k: round(v, 3) for k, v in by_family.items()},
                    activation_memory=memory, cpu_baseline=cpu, kernel_sweep=sweep, small_workloads=small)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
