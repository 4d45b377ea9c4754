"""Shared helpers of the GPU parity tests (test-side only)."""
import numpy as np

REL_L2_TOL = 1e-2      # stated tolerance for storage-precision attention outputs
MAX_ABS_TOL = 3e-2
TIE_BAND = 1e-4        # relative gap below which a selection boundary counts as a near tie


def to_dev(a, w, device="cuda:0"):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)
    return t if w.dtype == "f32" else t.to(torch.bfloat16)


def to_np(t):
    import torch
    if t.dtype == torch.bfloat16:
        t = t.float()
    return t.detach().cpu().numpy()


def storage_round(a, w):
    """Round an fp64 oracle array to the storage type, returned as float32."""
    from paper_2609_29812_b200.workloads import round_to_bf16
    a32 = np.asarray(a, dtype=np.float32)
    return a32 if w.dtype == "f32" else round_to_bf16(a32)


def attn_errors(got, ref):
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    return rel, float(np.max(np.abs(got - ref))) if got.size else 0.0


ERROR_LOG = []   # (what, carried roundings, relative L2, max abs, max-abs bound) of every attention comparison of the session


def half_ulp_storage(ref, bf16=True):
    """Largest rounding error of one store of a value as large as max|ref| in the storage type."""
    if not bf16:
        return 0.0
    mag = float(np.max(np.abs(ref))) if np.size(ref) else 0.0
    return 0.0 if mag == 0.0 else 2.0 ** (np.floor(np.log2(mag)) - 8)


def assert_attn_close(got, ref, what="", carried=0, bf16=True):
    """Relative L2 <= 1e-2 and max-abs <= 3e-2 (the stated tolerance) when both sides start from the same stored
    inputs.  `carried`: how many times the output carried into this comparison was rounded to the storage type on the
    GPU side only (the oracle carries fp64 between loops): the max-abs bound grows by half a storage ulp of the
    largest reference value per such rounding; the relative L2 bound stays as stated."""
    rel, mx = attn_errors(got, ref)
    bound = MAX_ABS_TOL + carried * half_ulp_storage(ref, bf16)
    ERROR_LOG.append((what, carried, float(rel), float(mx), float(bound)))
    assert rel <= REL_L2_TOL and mx <= bound, f"{what}: rel L2 {rel:.3e}, max abs {mx:.3e} (bound {bound:.3e})"
    return rel, mx


def assert_selection_matches(got_idx, ref_scores, cand, k, what=""):
    """`got_idx` (ascending ids) must equal the exact top-k of the fp64 `ref_scores` (aligned with `cand`)
    except inside a near-tie band around the boundary.  Returns the number of differing ids."""
    from oracle import flashloop_oracle as fo
    cand = np.asarray(cand, dtype=np.int64)
    ref_sel = fo.topk_ascending(ref_scores, k)
    ref_idx = cand[ref_sel]
    got_idx = np.asarray(got_idx, dtype=np.int64)
    assert len(got_idx) == len(ref_idx), what
    assert np.all(np.diff(got_idx) > 0), f"{what}: not strictly ascending"
    if np.array_equal(got_idx, ref_idx):
        return 0
    boundary = np.sort(ref_scores)[::-1][len(ref_idx) - 1]
    score_of = dict(zip(cand.tolist(), np.asarray(ref_scores, dtype=np.float64).tolist()))
    diff = np.setxor1d(got_idx, ref_idx)
    for j in diff:
        s = score_of[int(j)]
        assert abs(s - boundary) <= TIE_BAND * max(abs(boundary), 1e-300), \
            f"{what}: id {j} differs outside the near-tie band (score {s}, boundary {boundary})"
    return len(diff)
