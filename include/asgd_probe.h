/*
 * libasgd_probe -- issue-rate probes for sm_100a (a measuring aid of the K-Means ASGD library; the paper has no
 * counterpart).  The notes on the worker kernels quote what an instruction kind costs in issue slots on a B200;
 * this entry point measures those numbers on the GPU at hand.
 */
#ifndef ASGD_PROBE_H_
#define ASGD_PROBE_H_

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Cycles one of an SM's four schedulers spends per warp instruction (clock64 around unrolled loops, one block of
 * 16 warps per SM) for thirteen instruction streams, in this order:
 *   0 FFMA with two immediate operands      1 FFMA acc = x * w + acc (three registers)
 *   2 the packed two-wide FMA in that form  3 the packed two-wide add
 *   4 LOP3    5 FMNMX    6 FSET    7 IMAD   8 mma.sync m16n8k8 TF32 (the legacy tensor-core product)
 *   9 LOP3 and FFMA alternating            10 LOP3 and the packed FMA alternating
 *  11 one tensor-core product with six FFMA                12 one tensor-core product with four LOP3
 *   out_host     HOST [n_out], n_out >= 13 (written)
 *   scratch_dev  DEVICE, at least 4 * (1 + sms * 512) bytes, caller's; overwritten
 *   sms          blocks to launch (the GPU's SM count)
 * Launches on the default stream and synchronises.  Returns 0; -1 for a NULL pointer, n_out < 13 or sms < 1
 * (nothing is launched); -3 when a CUDA call failed.
 */
int asgd_probe_issue_rates(float *out_host, int n_out, float *scratch_dev, int sms);

/*
 * Cycles per tcgen05.mma (kind::f16, FP16 operands in shared memory with the 128-byte swizzle, M = 128, K = 16, fp32
 * accumulators in tensor memory), issued back to back by one thread of one block per SM (two threads in the last two
 * cases), twelve cases in this order:
 *   0 N = 256, the same pair of operand chunks every time     1 N = 256, walking over four chunks of each operand
 *   2 as 1 with a tcgen05.commit after every four products    3, 4, 5 the same three with N = 128
 *   6 as 2 with the commits going round eight barriers        7 as 2 with a fresh accumulator range after every commit
 *   8 as 1 with a commit after every 16 products              9 as 8 with the commits going round eight barriers
 *  10 two issuing threads (first lanes of two warps), each with its own accumulator range: four products and a
 *     commit in turn                                          11 the same without commits
 * These are the rates the tensor-core worker kernel's issuing threads can reach at best; cases 2 and 10 are why it
 * has two of them.
 *   out_host     HOST [n_out]; n_out >= 12: all cases, 6 <= n_out < 12: the first six (written)
 *   scratch_dev  DEVICE, at least 4 * sms bytes, caller's; overwritten
 *   sms          blocks to launch (the GPU's SM count)
 * Launches on the default stream and synchronises; every device-side wait is bounded.  Returns 0; -1 for a NULL
 * pointer, n_out < 6 or sms < 1 (nothing is launched); -3 when a CUDA call failed; -4 when a wait ran out.
 */
int asgd_probe_mma_rates(float *out_host, int n_out, float *scratch_dev, int sms);

#ifdef __cplusplus
}
#endif
#endif /* ASGD_PROBE_H_ */
