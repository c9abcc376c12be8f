"""The wide layer of the bench workload (65536 x 8192 x 8192, bf16) through the same calls the bench
times, checked on sampled outputs the oracle can compute one by one and on properties that hold at
any size.  Inputs come from the seeded generators; nothing here is compared with a stored value."""
import numpy as np
import pytest
import torch

from oracle import rad as orc
from workloads import layer_inputs, to_bf16_grid

from gpu_util import rel_err, to_host_f32

pytestmark = pytest.mark.gpu

B, D, H = 65536, 8192, 8192
P, SEED, LAYER, STEP = 0.1, 5, 1, 3
TILE_ROWS, TILE_COLS, TILE_WORDS, ALIGN = 64, 128, 288, 8


@pytest.fixture(scope="module")
def wide():
    import paper_2007_10412_b200 as rad
    A, dZ = layer_inputs(B, D, H, dtype="bf16", seed=77)
    rng = np.random.default_rng(78)
    W = to_bf16_grid(rng.standard_normal((D, H), dtype=np.float32) * np.float32(np.sqrt(2.0 / D)))
    bias = rng.standard_normal(H, dtype=np.float32)
    dev = dict(A=torch.from_numpy(A).to(torch.bfloat16).cuda(), dZ=torch.from_numpy(dZ).to(torch.bfloat16).cuda(),
               W=torch.from_numpy(W).to(torch.bfloat16).cuda(), bias=torch.from_numpy(bias).cuda())
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = rad.Store("different", "bf16", B, D, P, seed=SEED, layer=LAYER, step=STEP, relu_bits=False)
    rad.rad_linear_forward_store(dev["A"], st, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    yield dict(A=A, dZ=dZ, W=W, bias=bias, dev=dev, st=st, status=status, rad=rad)
    del dev, st
    torch.cuda.empty_cache()


def check_sampled_tiles(st, A, p, n_random=10, seed=1):
    """Keep bits, row offsets, tile extent and stored values of some tiles of a different-sample store of
    the wide layer, bit for bit against the oracle's definition evaluated on those tiles alone."""
    nslab, ncb = B // TILE_ROWS, D // TILE_COLS
    ntiles = nslab * ncb
    rng = np.random.default_rng(seed)
    tiles = [0, 1, ncb - 1, ncb, ntiles - 1, ntiles - ncb] + [int(t) for t in rng.integers(0, ntiles, n_random)]
    offsets = st.offsets.cpu().numpy().view(np.uint32)
    scale = np.float32(orc.scale_factor(p))
    for t in tiles:
        slab, blk = divmod(t, ncb)
        rows = np.arange(slab * TILE_ROWS, (slab + 1) * TILE_ROWS)
        cols = np.arange(blk * TILE_COLS, (blk + 1) * TILE_COLS)
        m = orc.keep_mask_at("different", rows, cols, p, SEED, LAYER, STEP)
        words = st.keepbits[t * TILE_WORDS:(t + 1) * TILE_WORDS].cpu().numpy().view(np.uint32)
        assert np.array_equal(words[:256], orc.pack_bits(m).reshape(-1)), t
        rowoff = np.concatenate([[0], np.cumsum(m.sum(axis=1))[:-1]]).astype(np.uint16)
        assert np.array_equal(words[256:].view(np.uint16), rowoff), t
        n = int(m.sum())
        padded = -(-n // ALIGN) * ALIGN
        assert int(offsets[t + 1]) - int(offsets[t]) == padded, t
        ref = orc.round_bf16(A[np.ix_(rows, cols)][m] * scale)
        got = st.values[int(offsets[t]):int(offsets[t]) + padded].view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(got[:n], orc.bf16_bits(ref)), t
        assert (got[n:] == 0).all(), t


def check_counts(st, p):
    """Identities that tie keep bits, offsets and the kept count together over the whole store."""
    ntiles = (B // TILE_ROWS) * (D // TILE_COLS)
    words = st.keepbits.view(ntiles, TILE_WORDS)[:, :256].contiguous()
    # set bits of every keep word, summed per tile on the device (lookups of a byte table)
    table = torch.tensor([bin(i).count("1") for i in range(256)], dtype=torch.int32, device="cuda")
    per_tile = torch.zeros(ntiles, dtype=torch.int64, device="cuda")
    for sh in (0, 8, 16, 24):
        per_tile += table[((words >> sh) & 0xFF).long()].sum(dim=1)
    nnz = st.nnz.cpu().numpy()
    assert int(per_tile.sum()) == int(nnz[0])
    offsets = st.offsets.cpu().numpy().view(np.uint32).astype(np.int64)
    assert offsets[0] == 0 and int(offsets[ntiles]) == int(nnz[1])
    padded = ((per_tile + (ALIGN - 1)) // ALIGN * ALIGN).cpu().numpy()
    assert np.array_equal(np.diff(offsets[:ntiles + 1]), padded)
    # Binomial(B D, p_eff): six standard deviations
    pe = orc.effective_p(p)
    assert abs(int(nnz[0]) - B * D * pe) < 6.0 * np.sqrt(B * D * pe * (1.0 - pe))


def check_weight_grad_entries(rad, st, A, dZ, dZ_dev, p, status, seed=2):
    """dW from a different-sample store of the wide layer on sampled (d, h) entries, each summed by the
    oracle over all 65536 rows from the mask and the rounded scaled values."""
    dW = torch.full((D, H), float("nan"), dtype=torch.float32, device="cuda")
    rad.rad_linear_weight_grad(st, dZ_dev, dW, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert torch.isfinite(dW).all()
    rng = np.random.default_rng(seed)
    ds = np.concatenate([[0, 127, 128, 255, 256, 511, 512, D - 1], rng.integers(0, D, 16)])
    hs = np.concatenate([[0, 255, 256, H - 1], rng.integers(0, H, 12)])
    scale = np.float32(orc.scale_factor(p))
    m = orc.keep_mask_at("different", np.arange(B), ds, p, SEED, LAYER, STEP)          # B x len(ds)
    a_hat = np.where(m, orc.round_bf16(A[:, ds] * scale), np.float32(0)).astype(np.float64)
    ref = a_hat.T @ dZ[:, hs].astype(np.float64)
    got = to_host_f32(dW[torch.from_numpy(ds).cuda()][:, torch.from_numpy(hs).cuda()])
    fro, mx = rel_err(got, ref)
    assert fro <= 2e-2 and mx <= 2e-2, (fro, mx)
    # float32 accumulation of exact bf16 products: far inside the stated tolerance
    bound = 1e-4 * (np.abs(a_hat).T @ np.abs(dZ[:, hs]).astype(np.float64))
    assert (np.abs(got - ref) <= bound + 1e-30).all()
    del dW


def test_store_sampled_tiles_are_bit_exact(wide):
    check_sampled_tiles(wide["st"], wide["A"], P)


@pytest.mark.parametrize("p", [0.01, 0.05, 0.5])
def test_store_and_weight_grad_over_the_p_sweep(wide, p):
    """The other keep probabilities the bench sweeps: the pipelined store on sampled tiles and count
    identities; at p = 0.5 also dW, whose expander then takes its dense-word path."""
    rad, status = wide["rad"], wide["status"]
    st = rad.Store("different", "bf16", B, D, p, seed=SEED, layer=LAYER, step=STEP, relu_bits=False)
    rad.rad_linear_forward_store(wide["dev"]["A"], st, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    check_sampled_tiles(st, wide["A"], p, n_random=6, seed=int(p * 1000))
    check_counts(st, p)
    if p == 0.5:
        check_weight_grad_entries(rad, st, wide["A"], wide["dZ"], wide["dev"]["dZ"], p, status, seed=9)
    del st
    torch.cuda.empty_cache()


@pytest.mark.parametrize("p", [0.01, 0.1, 0.5])
def test_same_sample_store_and_weight_grad(wide, p):
    """Same-sample variant at the size the bench times it (Sec. 4.3: one mask for the whole minibatch): the
    kept-column list and keep bits in full, sampled rows of the gathered block bit for bit, zero fill beyond
    the kept count; dW on sampled entries of kept rows, and exactly zero on every row that was not kept."""
    rad, status, A, dZ = wide["rad"], wide["status"], wide["A"], wide["dZ"]
    st = rad.Store("same", "bf16", B, D, p, seed=SEED, layer=LAYER, step=STEP, relu_bits=False)
    rad.rad_linear_forward_store(wide["dev"]["A"], st, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    m = orc.keep_mask_at("same", [0], np.arange(D), p, SEED, LAYER, STEP)[0]
    idx = np.flatnonzero(m)
    k = idx.size
    nnz = st.nnz.cpu().numpy()
    assert nnz[0] == k and nnz[1] == k * B
    assert np.array_equal(st.offsets[:k].cpu().numpy().view(np.uint32), idx.astype(np.uint32))
    assert np.array_equal(st.keepbits.cpu().numpy().view(np.uint32), orc.pack_bits(m[None, :]).reshape(-1))
    ld = int(st.c.values_ld)
    rng = np.random.default_rng(6)
    bs = np.concatenate([[0, 1, 63, 64, 127, 128, B - 1], rng.integers(0, B, 25)])
    got = st.values.view(B, ld)[torch.from_numpy(bs).cuda()].view(torch.int16).cpu().numpy().view(np.uint16)
    scale = np.float32(orc.scale_factor(p))
    ref = orc.bf16_bits(orc.round_bf16(A[np.ix_(bs, idx)] * scale))
    assert np.array_equal(got[:, :k], ref)
    assert (got[:, k:] == 0).all()
    # weight gradient from the store
    dW = torch.full((D, H), float("nan"), dtype=torch.float32, device="cuda")
    rad.rad_linear_weight_grad(st, wide["dev"]["dZ"], dW, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    kept = torch.from_numpy(m).cuda()
    assert (dW[~kept] == 0).all()                       # rows of columns that were not kept: exactly zero
    assert torch.isfinite(dW[kept]).all()
    ds = np.concatenate([idx[[0, 1, k // 2, k - 1]], rng.choice(idx, 12)])
    hs = np.concatenate([[0, 255, 256, H - 1], rng.integers(0, H, 12)])
    a_c = orc.round_bf16(A[:, ds] * scale).astype(np.float64)
    ref = a_c.T @ dZ[:, hs].astype(np.float64)
    got = to_host_f32(dW[torch.from_numpy(ds).cuda()][:, torch.from_numpy(hs).cuda()])
    fro, mx = rel_err(got, ref)
    assert fro <= 2e-2 and mx <= 2e-2, (fro, mx)
    bound = 1e-4 * (np.abs(a_c).T @ np.abs(dZ[:, hs]).astype(np.float64))
    assert (np.abs(got - ref) <= bound + 1e-30).all()
    del st, dW
    torch.cuda.empty_cache()


def test_store_counts_hold_together(wide):
    check_counts(wide["st"], P)


def test_weight_grad_sampled_entries(wide):
    check_weight_grad_entries(wide["rad"], wide["st"], wide["A"], wide["dZ"], wide["dev"]["dZ"], P, wide["status"])


def test_store_without_held_keep_bits_at_full_size(wide):
    """The variant that holds no keep bits, through the pipelined store with its index in the workspace and the
    index drawn again for dW: the same offsets, counts and values as the store that holds its index (which the
    tests above check against the oracle), dW on the oracle's sampled entries and identical to the other dW."""
    rad, dev, status = wide["rad"], wide["dev"], wide["status"]
    held = rad.Store("redrawn", "bf16", B, D, P, seed=SEED, layer=LAYER, step=STEP, relu_bits=False)
    assert held.keepbits.numel() == 0
    rad.rad_linear_forward_store(dev["A"], held, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    full = wide["st"]
    assert torch.equal(held.offsets, full.offsets) and torch.equal(held.nnz, full.nnz)
    used = int(full.nnz.cpu()[1])
    assert torch.equal(held.values[:used].view(torch.int16), full.values[:used].view(torch.int16))
    check_weight_grad_entries(rad, held, wide["A"], wide["dZ"], dev["dZ"], P, status)
    dW_a = torch.empty(D, H, dtype=torch.float32, device="cuda")
    dW_b = torch.empty(D, H, dtype=torch.float32, device="cuda")
    rad.rad_linear_weight_grad(held, dev["dZ"], dW_a, dev_status=status)
    rad.rad_linear_weight_grad(full, dev["dZ"], dW_b, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0 and torch.equal(dW_a, dW_b)
    del dW_a, dW_b, held


def test_forward_and_input_grad_sampled_entries(wide):
    rad, dev, A, W, bias, dZ = wide["rad"], wide["dev"], wide["A"], wide["W"], wide["bias"], wide["dZ"]
    act = torch.empty(B, H, dtype=torch.bfloat16, device="cuda")
    zlow = torch.empty(B, H, dtype=torch.bfloat16, device="cuda")
    rad.rad_linear_forward(dev["A"], dev["W"], dev["bias"], "gelu", out_act=act, out_zlow=zlow, dev_status=wide["status"])
    torch.cuda.synchronize()
    assert wide["status"].item() == 0
    rng = np.random.default_rng(3)
    bs = np.concatenate([[0, 127, 128, 255, 256, B - 1], rng.integers(0, B, 18)])
    hs = np.concatenate([[0, 127, 128, 255, 256, H - 1], rng.integers(0, H, 10)])
    z = A[bs].astype(np.float64) @ W[:, hs].astype(np.float64) + bias[hs]
    bi, hi = torch.from_numpy(bs).cuda(), torch.from_numpy(hs).cuda()
    assert max(rel_err(to_host_f32(zlow[bi][:, hi]), z)) <= 8e-3
    assert max(rel_err(to_host_f32(act[bi][:, hi]), orc.act_forward(z, "gelu"))) <= 8e-3
    del act
    # input gradient with the GELU derivative taken at the stored pre-activation
    dA = torch.empty(B, D, dtype=torch.bfloat16, device="cuda")
    db = torch.empty(H, dtype=torch.float32, device="cuda")
    zprev = dev["A"]                                   # any B x D bf16 tensor serves as the pre-activation
    rad.rad_linear_input_grad(dev["dZ"], dev["W"], z_prev=zprev, dZ_prev=dA, db=db, dev_status=wide["status"])
    torch.cuda.synchronize()
    assert wide["status"].item() == 0
    ds = np.concatenate([[0, 127, 128, 255, 256, D - 1], rng.integers(0, D, 10)])
    g = dZ[bs].astype(np.float64) @ W[ds].astype(np.float64).T                       # len(bs) x len(ds)
    ref = orc.round_bf16((g * orc.gelu_grad(A[np.ix_(bs, ds)].astype(np.float64))).astype(np.float32)).astype(np.float64)
    got = to_host_f32(dA[bi][:, torch.from_numpy(ds).cuda()])
    assert max(rel_err(got, ref)) <= 2e-2
    ref_db = dZ[:, hs].astype(np.float64).sum(axis=0)
    assert max(rel_err(to_host_f32(db[hi]), ref_db)) <= 1e-5


def test_fused_forward_fills_the_next_store(wide):
    """The forward GEMM of the wide layer with the next layer's store filled from its epilogue: sampled
    tiles of that store against the oracle's rule applied to the activations the same call wrote, and the
    count identities over the whole store."""
    rad, dev, status = wide["rad"], wide["dev"], wide["status"]
    act = torch.empty(B, H, dtype=torch.bfloat16, device="cuda")
    st = rad.Store("different", "bf16", B, H, P, seed=SEED, layer=LAYER + 1, step=STEP, relu_bits=False)
    st.values.fill_(float("nan"))
    rad.rad_linear_forward_fill(dev["A"], dev["W"], dev["bias"], "gelu", act, st, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    check_counts(st, P)
    nslab, ncb = B // TILE_ROWS, H // TILE_COLS
    ntiles = nslab * ncb
    rng = np.random.default_rng(11)
    offsets = st.offsets.cpu().numpy().view(np.uint32)
    scale = np.float32(orc.scale_factor(P))
    for t in [0, ncb - 1, ntiles - 1, ntiles - ncb] + [int(t) for t in rng.integers(0, ntiles, 8)]:
        slab, blk = divmod(t, ncb)
        rows = np.arange(slab * TILE_ROWS, (slab + 1) * TILE_ROWS)
        cols = np.arange(blk * TILE_COLS, (blk + 1) * TILE_COLS)
        m = orc.keep_mask_at("different", rows, cols, P, SEED, LAYER + 1, STEP)
        words = st.keepbits[t * TILE_WORDS:(t + 1) * TILE_WORDS].cpu().numpy().view(np.uint32)
        assert np.array_equal(words[:256], orc.pack_bits(m).reshape(-1)), t
        n = int(m.sum())
        padded = -(-n // ALIGN) * ALIGN
        assert int(offsets[t + 1]) - int(offsets[t]) == padded, t
        a_tile = to_host_f32(act[slab * TILE_ROWS:(slab + 1) * TILE_ROWS, blk * TILE_COLS:(blk + 1) * TILE_COLS])
        ref = orc.round_bf16(a_tile[m] * scale)
        got = st.values[int(offsets[t]):int(offsets[t]) + padded].view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(got[:n], orc.bf16_bits(ref)), t
        assert (got[n:] == 0).all(), t
    del st, act
    torch.cuda.empty_cache()


@pytest.mark.parametrize("law", ["replace", "fixed"])
def test_other_sampling_laws_sampled_tiles_and_counts(wide, law):
    """The with-replacement and the fixed-count law at the size the bench sweep times them: sampled store
    tiles bit for bit against the oracle (multiplicities of the tile's 64 rows over all columns), offsets
    against the keep-bit population, and the kept count (exactly B k without replacement)."""
    rad, A = wide["rad"], wide["A"]
    st = rad.Store("different", "bf16", B, D, P, seed=SEED, layer=LAYER, step=STEP, relu_bits=False, law=law)
    status = wide["status"]
    rad.rad_linear_forward_store(wide["dev"]["A"], st, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    nslab, ncb = B // TILE_ROWS, D // TILE_COLS
    ntiles = nslab * ncb
    k = orc.draws_per_row(P, D)
    s = orc.replace_scale(P, D)
    offsets = st.offsets.cpu().numpy().view(np.uint32).astype(np.int64)
    nnz = st.nnz.cpu().numpy()
    count = orc.multiplicity if law == "replace" else orc.fixed_subset
    rng = np.random.default_rng(4)
    for t in [0, ncb - 1, ntiles - 1] + [int(t) for t in rng.integers(0, ntiles, 5)]:
        slab, blk = divmod(t, ncb)
        rows = np.arange(slab * TILE_ROWS, (slab + 1) * TILE_ROWS)
        c_rows = count("different", B, D, P, SEED, LAYER, STEP, rows=rows)
        assert (c_rows.sum(axis=1) == k).all()
        c = c_rows[:, blk * TILE_COLS:(blk + 1) * TILE_COLS]
        m = c > 0
        words = st.keepbits[t * TILE_WORDS:(t + 1) * TILE_WORDS].cpu().numpy().view(np.uint32)
        assert np.array_equal(words[:256], orc.pack_bits(m).reshape(-1)), t
        rowoff = np.concatenate([[0], np.cumsum(m.sum(axis=1))[:-1]]).astype(np.uint16)
        assert np.array_equal(words[256:].view(np.uint16), rowoff), t
        n = int(m.sum())
        padded = -(-n // ALIGN) * ALIGN
        assert offsets[t + 1] - offsets[t] == padded, t
        tile = A[np.ix_(rows, np.arange(blk * TILE_COLS, (blk + 1) * TILE_COLS))]
        ref = orc.round_bf16(tile * (c.astype(np.float32) * s))[m]
        got = st.values[int(offsets[t]):int(offsets[t]) + padded].view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(got[:n], orc.bf16_bits(ref)), t
        assert (got[n:] == 0).all(), t
    words = st.keepbits.view(ntiles, TILE_WORDS)[:, :256].contiguous()
    table = torch.tensor([bin(i).count("1") for i in range(256)], dtype=torch.int32, device="cuda")
    per_tile = torch.zeros(ntiles, dtype=torch.int64, device="cuda")
    for sh in (0, 8, 16, 24):
        per_tile += table[((words >> sh) & 0xFF).long()].sum(dim=1)
    assert int(per_tile.sum()) == int(nnz[0]) and int(offsets[ntiles]) == int(nnz[1])
    if law == "fixed":
        assert int(nnz[0]) == B * k
    else:
        mean = B * D * (1.0 - (1.0 - 1.0 / D) ** k)
        assert abs(int(nnz[0]) - mean) < 6.0 * np.sqrt(mean)      # the distinct count varies less than a Poisson
    del st
    torch.cuda.empty_cache()


def test_projection_sampled_entries(wide):
    """The random projection at the bench size: S = A R' on sampled rows and dW_hat = R' ((S^T dZ) / k) on
    sampled entries against the oracle's definition (S over all rows in float32: bf16 inputs and signs give
    exact products)."""
    rad, A, dZ = wide["rad"], wide["A"], wide["dZ"]
    st = rad.Store("project", "bf16", B, D, P, seed=SEED, layer=LAYER, step=STEP, relu_bits=False)
    status = wide["status"]
    rad.rad_linear_forward_store(wide["dev"]["A"], st, status)
    dW = torch.empty(D, H, dtype=torch.float32, device="cuda")
    ws = torch.empty(max(rad.rad_weight_grad_workspace(st, H), 256), dtype=torch.uint8, device="cuda")
    rad.rad_linear_weight_grad(st, wide["dev"]["dZ"], dW, ws, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    k = orc.draws_per_row(P, D)
    assert st.nnz.cpu().numpy()[0] == k
    R = orc.rademacher(D, k, SEED, LAYER, STEP).astype(np.float32)
    S = np.empty((B, k), dtype=np.float32)
    for b0 in range(0, B, 8192):
        S[b0:b0 + 8192] = orc.round_bf16(A[b0:b0 + 8192] @ R)
    ld = st.c.values_ld
    rng = np.random.default_rng(5)
    bs = np.concatenate([[0, 127, 128, B - 1], rng.integers(0, B, 28)])
    got_S = to_host_f32(st.values.view(B, ld)[torch.from_numpy(bs).cuda()])
    assert (got_S[:, k:] == 0).all()
    assert max(rel_err(got_S[:, :k], S[bs])) <= 8e-3
    hs = np.concatenate([[0, 255, 256, H - 1], rng.integers(0, H, 12)])
    ds = np.concatenate([[0, 255, 256, D - 1], rng.integers(0, D, 12)])
    G = (S.astype(np.float64).T @ dZ[:, hs].astype(np.float64)).astype(np.float32) * (np.float32(1.0) / np.float32(k))
    ref = R[ds].astype(np.float64) @ orc.round_bf16(G).astype(np.float64)
    got = to_host_f32(dW[torch.from_numpy(ds).cuda()][:, torch.from_numpy(hs).cuda()])
    assert max(rel_err(got, ref)) <= 2e-2
    del st, dW, ws
    torch.cuda.empty_cache()
