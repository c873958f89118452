/* CPU oracle for the Tetra encoder's search -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * For a block of 24 weights the encoder looks for the point of the format's
 * codebook whose direction is closest to the block, and picks the gain bit
 * (Sec. 3.1, Eq. (2)).  The paper's own search is not exhaustive and is not
 * specified (two trial scales, a few candidates per section joined over the
 * trellis, Sec. 3.1); what IS fixed is the objective and the codebook, so this
 * oracle computes the exact optimum:
 *
 *     maximise  <w, y> / (|w| |y|)  over every 47-bit index (all paths, both
 *     parities, both classes, all rows of the lists) with y != 0,
 *
 * then the gain bit that minimises |w - y/|y| gain[g] sigma|^2.  It exploits
 * that the codebook is a product of three sections tied by the trellis path, the
 * parity and Eq. (3): per section, pattern byte, class and section norm only the
 * best correlation matters, and the three sections are joined state by state
 * with the summed norm and the class parity as extra state.  Every candidate
 * of a section is produced by the decoder's own to_decode_section.
 *
 * Readings: E1 the objective is the cosine (scale-free), ties go to the first
 * candidate in (parity, state, branch, class, norm) order; E2 the gain bit is
 * argmin_g (gain[g] sigma)^2 - 2 gain[g] sigma <w,y>/|y|; E3 a zero block
 * encodes as the all-zero word.
 *
 * Pins (tests/test_encode_oracle_pins.py): brute force over the whole codebook
 * restricted to the first few rows of every list, through to_decode_word;
 * decode -> encode round trips (cosine 1); never worse than sampled codewords;
 * the retention of Sec. 3.5 on Gaussian blocks lies between the paper's
 * figure for its non-exhaustive search and the figure of the 24-dimensional
 * ball; the gain rule against a direct evaluation of the error.  Two pins that
 * do not share this search's decomposition, both through to_decode_word only:
 * planted optima (codebook points from deep rows -- ranks 2 to 4, the class-1
 * half of the middle list, both parities -- turned by 3 degrees, where any two
 * codebook directions are at least 15.9 degrees apart, must come back as the
 * planted direction), and a brute-force neighbourhood (none of the ~10,000
 * words that differ from the answer in one field has a larger cosine; over a
 * million words in all).
 */
#ifndef TETRA_ENCODE_ORACLE_H
#define TETRA_ENCODE_ORACLE_H
#include "tetra_oracle.h"

/* row_limit: 2048 for the format's lists; smaller values restrict every list
 * (per class) to its first row_limit entries, for the brute-force pin.
 * Returns 0 and writes the 47-bit index (gain bit 0) and the cosine; -1 if
 * row_limit is out of range. */
int to_encode_block(const to_tables *t, const double w[24], int row_limit, uint64_t *word, double *cosine);

/* Gain bit for a block with correlation c = <w,y>/|y| (reading E2). */
int to_choose_gain(double c, double sigma, const double gain[2]);

/* n blocks (w: n x 24), OpenMP over blocks; words carry the gain bit chosen with
 * (sigma, gain). */
int to_encode_blocks(const to_tables *t, const double *w, size_t n, int row_limit, double sigma,
                     const double gain[2], uint64_t *words, double *cosines, int threads);
#endif
